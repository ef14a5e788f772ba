// Fused base + multi-LoRA GEMM on the sm_100a tensor cores (Sec. 3.1: y = xW + sum_a s_a (xA_a)B_a).
//
//   y[128 x BN tile] = x_tile W^T_tile                        (K/64 pipeline stages, 4 UMMAs each)
//                    + sum over the tile's LoRA slabs  t_slab B_slab   (one K=16 UMMA per slab,
//                      into the SAME TMEM accumulator)
//                    -> epilogue: bias, GELU / residual / patch-embed placement, bf16 store.
//
// t (the scaled, row-masked shrink x A_cat of the tile) is produced by launch_shrink before the
// GEMM and fetched by TMA like any other operand.  Operands are staged by TMA into 128B- (base)
// and 32B- (LoRA slab) swizzled shared memory; a single thread issues tcgen05.mma; accumulators
// live in TMEM (two buffers, so the epilogue of one tile overlaps the main loop of the next).
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..9 = epilogue (two
// warps per TMEM lane quarter, each taking half of the tile's columns).
// Every mbarrier wait is bounded: on expiry the CTA raises an abort flag, records
// PM_ERR_TIMEOUT in the status word, drains and returns.
// When n_out is a multiple of 256 the CTA-pair variant (lora_gemm_pair_kernel, cta_group::2, 256 x 256
// tiles) is used; the single-CTA kernel serves the narrower shapes.
#include "common.cuh"
#include "tcgen05_ptx.cuh"

#define BUMP(L) do { if ((L).launches) ++*(L).launches; } while (0)

namespace {

constexpr int BM = PM_TILE_M;
constexpr int BK = 64;
constexpr int STAGES = 4;
constexpr int SHRINK_THREADS = 192;
constexpr int SLABS_PER_STAGE = 4;

// Exact-erf GELU x * Phi(x), evaluated in logistic form: Phi(x) = 1 / (1 + exp(-2 x p(x^2))) holds
// exactly for p = atanh(erf(x / sqrt 2)) / x, which a quadratic in x^2 fits well enough that
//   | x (1/2 + 1/2 tanh(x q(x^2))) - gelu(x) | < 2.6e-5   for all x     (q = p: 1 / (1 + e^-2u) = 1/2 + 1/2 tanh u),
// far below the bf16 rounding of the stored result except where the result itself is below 1e-2; the
// hardware tanh (tanh.approx.f32, relative error about 2^-11) adds less than a quarter of a bf16 step.
// The epilogue warps share their issue slots with the thread that issues the MMAs, so every
// instruction saved here counts: the arithmetic runs on pairs (packed fp32) and costs one special-function
// instruction per element (the form x / (1 + 2^(x q)) it replaces needed an exponential and a
// reciprocal: fused GEMMs 2.3 % slower in the bench step).

// Two fp32 values in one 64-bit register, for the packed fp32 arithmetic of sm_100 (one issue slot
// for two results; each half is the ordinary IEEE operation).
__device__ __forceinline__ uint64_t pk2(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void upk2(uint64_t r, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// the GELU described above, on a pair
__device__ __forceinline__ uint64_t gelu_erf2(uint64_t v) {
    // v^2 is capped where Phi has long saturated (the fitted q turns over beyond |v| = 7.2)
    float t0, t1;
    upk2(mul2(v, v), t0, t1);
    const uint64_t t = pk2(fminf(t0, 50.f), fminf(t1, 50.f));
    uint64_t q = fma2(t, pk2(-3.5151945e-04f, -3.5151945e-04f), pk2(3.7005664e-02f, 3.7005664e-02f));
    q = fma2(q, t, pk2(0.79750784f, 0.79750784f));
    float w0, w1, h0, h1;
    upk2(mul2(v, q), w0, w1);
    asm("tanh.approx.f32 %0, %1;" : "=f"(h0) : "f"(w0));
    asm("tanh.approx.f32 %0, %1;" : "=f"(h1) : "f"(w1));
    return mul2(v, fma2(pk2(h0, h1), pk2(0.5f, 0.5f), pk2(0.5f, 0.5f)));
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}

struct GemmArgs {
    int rows, k_in, n_out, m_tiles, n_tiles, epi;
    const float* bias;
    const bf16* residual;
    bf16* y;
    PatchEpi pe;
    // LoRA plan (null tile_nslabs = no LoRA)
    const int* tile_nslabs;
    const int* tile_slab;
    int slab_cap;
    int tma_store;             // 1: the epilogue stores through shared memory + TMA (tm_y valid)
    int overlap_prev;          // host side only: launch with programmatic serialization (the kernel before it on
                               // the stream is this linear's shrink, whose results are awaited with dep_wait())
    int* status;
    // LayerNorm folded into the linear (LNF kernels): y = rstd (acc - mean g) + bias, per row / column
    const float* ln_g;
    const float2* ln_stats;
};

constexpr int STAGING_BYTES_PER_WARP = 2 * 32 * 64;     // two [32 rows x 32 bf16] buffers
constexpr int PLAN_BYTES = 2048;

// EW = number of epilogue warps (4 or 8); the CTA has 2 + EW warps.
template <int BN, int EW>
struct Smem {
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int T_SLAB_BYTES = BM * PM_SLAB * 2;      // 4096
    static constexpr int B_SLAB_BYTES = BN * PM_SLAB * 2;
    static constexpr int STAGING_OFFSET = STAGES * STAGE_BYTES;
    static constexpr int PLAN_OFFSET = STAGING_OFFSET + EW * STAGING_BYTES_PER_WARP;
    static constexpr int BAR_OFFSET = PLAN_OFFSET + PLAN_BYTES;
    static constexpr int TOTAL = BAR_OFFSET + 256;             // + barriers (base must be 1024-aligned)
};

// Epilogue of one 128 x BN accumulator by one epilogue warp: its share of the tile's 32-column
// chunks goes TMEM -> registers -> bias / GELU / residual / patch placement -> bf16 -> shared
// memory -> TMA store (or straight to global memory).  Returns false once the CTA is aborting.
// PAIR: the accumulator-free barrier lives in the even CTA of a pair (tempty_addr is a cluster address).
// RES_SMEM: the residual rows come through shared memory (TMA into res_buf, four 2 KB chunks of this
// warp, completion on res_bar) instead of per-thread global loads.
template <int BN, int EPI, int HALVES, bool PAIR, bool LNF, bool RES_SMEM>
__device__ __forceinline__ bool epilogue_tile(const GemmArgs& args, const CUtensorMap& tm_y, uint32_t staging,
                                              uint32_t& chunk_no, uint32_t tmem_base, int acc, uint32_t acc_phase,
                                              uint32_t tfull_addr, uint32_t tempty_addr, volatile int* abort_flag,
                                              int m, int n, int quarter, int half, int lane,
                                              const CUtensorMap* tm_res, uint32_t res_buf, uint32_t res_bar,
                                              uint32_t res_phase) {
    constexpr int CPW = BN / 32 / HALVES;         // 32-column chunks per epilogue warp
    const int row = m * BM + quarter * 32 + lane;     // m: 128-row tile index
    const bool row_ok = row < args.rows;
    const int n_chunks = min(BN / 32, (args.n_out - n * BN) / 32);      // even: n_out % 64 == 0
    const int my_chunks = n_chunks / HALVES;
    const int c0 = half * my_chunks;
    // The residual rows of this warp's chunks are fetched before the accumulator is ready, so
    // their latency hides behind the main loop.  (In-place use, y == residual, is safe: the
    // same thread reads an element here and is the only one to overwrite it below.)
    uint4 rr[(EPI == EPI_RESIDUAL && !RES_SMEM) ? CPW : 1][4];
    if constexpr (EPI == EPI_RESIDUAL && RES_SMEM) {
        // one thread asks TMA for this warp's chunks of the residual tile (rows past the end read as
        // zero); the warp's reads of the previous tile's chunks are ordered before these writes
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
            mbar_expect_tx(res_bar, (uint32_t)(my_chunks * 32 * 64));
            for (int cc = 0; cc < my_chunks; ++cc)
                tma_load_2d(res_buf + cc * (32 * 64), tm_res, n * BN + (c0 + cc) * 32, m * BM + quarter * 32, res_bar);
        }
    } else if constexpr (EPI == EPI_RESIDUAL) {
#pragma unroll
        for (int cc = 0; cc < CPW; ++cc) {
            if (cc < my_chunks && row_ok) {
                const uint4* r4 = reinterpret_cast<const uint4*>(
                    args.residual + (size_t)row * args.n_out + n * BN + (c0 + cc) * 32);
#pragma unroll
                for (int q = 0; q < 4; ++q) rr[cc][q] = r4[q];
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q) rr[cc][q] = make_uint4(0, 0, 0, 0);
            }
        }
    }
    bool ok = PAIR ? mbar_wait_cluster(tfull_addr, acc_phase, abort_flag, args.status)
                   : mbar_wait(tfull_addr, acc_phase, abort_flag, args.status);
    ok = __all_sync(0xFFFFFFFFu, ok);
    if (!ok) return false;
    tc_fence_after();
    size_t orow = (size_t)row;
    const float* pos_row = nullptr;
    if (EPI == EPI_PATCH && row_ok) {
        const int p = row % args.pe.g2;
        orow = (size_t)(row / args.pe.g2) * args.pe.tokens + 1 + p;
        pos_row = args.pe.pos + (size_t)(1 + p) * args.n_out;
    }
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
    float2 st = make_float2(0.f, 1.f);                 // (mean, rstd) of this thread's row
    if (LNF && row_ok) st = args.ln_stats[row];
#pragma unroll
    for (int cc = 0; cc < CPW; ++cc) {
        if (cc >= my_chunks) break;
        const int c = c0 + cc;
        const int n0 = n * BN + c * 32;
        uint32_t v[32];
        tmem_ld32(t_row + (uint32_t)(c * 32), v);
        tmem_ld_wait();
        if (cc == my_chunks - 1) {
            // every TMEM read of this accumulator is done: hand the buffer back early
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { if (PAIR) mbar_arrive_cluster(tempty_addr); else mbar_arrive(tempty_addr); }
        }
        // bias (and the folded LayerNorm: rstd (acc - mean g) + b) and GELU, two columns per instruction
        uint64_t fp[16];                                 // columns (2i, 2i+1) of this chunk
        const uint64_t rstd2 = pk2(st.y, st.y), nmean2 = pk2(-st.x, -st.x);
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
            const float4 b4 = __ldg(reinterpret_cast<const float4*>(args.bias + n0 + j));
            uint64_t a0 = pk2(__uint_as_float(v[j + 0]), __uint_as_float(v[j + 1]));
            uint64_t a1 = pk2(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
            if constexpr (LNF) {
                const float4 g4 = __ldg(reinterpret_cast<const float4*>(args.ln_g + n0 + j));
                a0 = fma2(rstd2, fma2(nmean2, pk2(g4.x, g4.y), a0), pk2(b4.x, b4.y));
                a1 = fma2(rstd2, fma2(nmean2, pk2(g4.z, g4.w), a1), pk2(b4.z, b4.w));
            } else {
                a0 = add2(a0, pk2(b4.x, b4.y));
                a1 = add2(a1, pk2(b4.z, b4.w));
            }
            if constexpr (EPI == EPI_GELU) { a0 = gelu_erf2(a0); a1 = gelu_erf2(a1); }
            fp[j >> 1] = a0;
            fp[(j >> 1) + 1] = a1;
        }
        if constexpr (EPI == EPI_RESIDUAL) {
            if constexpr (RES_SMEM) {
                if (cc == 0) {
                    ok = mbar_wait(res_bar, res_phase, abort_flag, args.status);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) return false;
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint4 r4v;
                if constexpr (RES_SMEM) {
                    // same 64B swizzle as the store staging: 16-byte chunk q of row `lane`
                    const uint32_t a = res_buf + cc * (32 * 64) + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4);
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(r4v.x), "=r"(r4v.y), "=r"(r4v.z), "=r"(r4v.w) : "r"(a));
                } else {
                    r4v = rr[cc][q];
                }
                const uint32_t w[4] = {r4v.x, r4v.y, r4v.z, r4v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    fp[q * 4 + e] = add2(fp[q * 4 + e], pk2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xFFFF0000u)));
            }
        } else if constexpr (EPI == EPI_PATCH) {
            if (row_ok) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float4 p4 = __ldg(reinterpret_cast<const float4*>(pos_row + n0 + j));
                    fp[j >> 1] = add2(fp[j >> 1], pk2(p4.x, p4.y));
                    fp[(j >> 1) + 1] = add2(fp[(j >> 1) + 1], pk2(p4.z, p4.w));
                }
            }
        }
        uint4 o[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float lo, hi;
            upk2(fp[q * 4 + 0], lo, hi); o[q].x = pack_bf16(lo, hi);
            upk2(fp[q * 4 + 1], lo, hi); o[q].y = pack_bf16(lo, hi);
            upk2(fp[q * 4 + 2], lo, hi); o[q].z = pack_bf16(lo, hi);
            upk2(fp[q * 4 + 3], lo, hi); o[q].w = pack_bf16(lo, hi);
        }
        if (args.tma_store) {
            // [32 rows x 64 B] block, 16-byte chunks XOR-swizzled by (row >> 1) & 3 (64B
            // swizzle), then one TMA store; rows past the end are clipped by the tensor map
            const uint32_t buf = staging + (chunk_no & 1u) * (32 * 64);
            if (lane == 0) bulk_wait_read1();        // the store that last used this buffer has read it
            __syncwarp();
#pragma unroll
            for (int q = 0; q < 4; ++q)
                st_shared_v4(buf + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4), o[q]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                tma_store_2d(&tm_y, buf, n0, m * BM + quarter * 32);
                bulk_commit();
            }
            ++chunk_no;
        } else if (row_ok) {
            uint4* o4 = reinterpret_cast<uint4*>(args.y + orow * args.n_out + n0);
#pragma unroll
            for (int q = 0; q < 4; ++q) o4[q] = o[q];
        }
    }
    return true;
}

template <int BN, int EPI, int EW, bool LNF>
__global__ void __launch_bounds__(64 + 32 * EW, 1)
lora_gemm_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                 const __grid_constant__ CUtensorMap tm_t, const __grid_constant__ CUtensorMap tm_bt,
                 const __grid_constant__ CUtensorMap tm_y, const GemmArgs args) {
    using S = Smem<BN, EW>;
    constexpr int NTHREADS = 64 + 32 * EW;
    constexpr int HALVES = EW / 4;                // epilogue warps per TMEM lane quarter
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if (base & 1023u) {                       // swizzled operands need a 1024-byte aligned window
        if (threadIdx.x == 0) atomicCAS(args.status, 0, (int)PM_ERR_CUDA);
        return;
    }
    uint8_t* smem = smem_raw;
    const uint32_t bars = base + S::BAR_OFFSET;
    // barrier words: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto tfull_bar = [&](int s) { return bars + 8u * (2 * STAGES + s); };
    auto tempty_bar = [&](int s) { return bars + 8u * (2 * STAGES + 2 + s); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + S::BAR_OFFSET + 8 * (2 * STAGES + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::BAR_OFFSET + 8 * (2 * STAGES + 4) + 8);
    int* plan = reinterpret_cast<int*>(smem + S::PLAN_OFFSET);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = args.m_tiles * args.n_tiles;
    const int num_kb = args.k_in / BK;

    // The LoRA plan of this CTA's tiles (slab count + arena slab ids) is copied to shared memory
    // once, so that the producer and the MMA issuer never wait on a global load between tiles.
    const int plan_stride = 1 + args.slab_cap;
    const int plan_tiles = args.tile_nslabs ? PLAN_BYTES / (4 * plan_stride) : 0;
    if (args.tile_nslabs) {
        for (int i = threadIdx.x / 8; i < plan_tiles; i += NTHREADS / 8) {
            const int tile = blockIdx.x + i * gridDim.x;
            if (tile >= total_tiles) break;
            const int m = tile / args.n_tiles;
            const int ns = args.tile_nslabs[m];
            if ((threadIdx.x & 7) == 0) plan[i * plan_stride] = ns;
            for (int q = threadIdx.x & 7; q < ns; q += 8) plan[i * plan_stride + 1 + q] = args.tile_slab[m * args.slab_cap + q];
        }
    }
    auto tile_ns = [&](int it, int m) -> int {
        if (!args.tile_nslabs) return 0;
        return it < plan_tiles ? plan[it * plan_stride] : args.tile_nslabs[m];
    };
    auto tile_slab_id = [&](int it, int m, int q) -> int {
        return it < plan_tiles ? plan[it * plan_stride + 1 + q] : args.tile_slab[m * args.slab_cap + q];
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(tfull_bar(s), 1); mbar_init(tempty_bar(s), EW); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32((const void*)tmem_slot), 2 * BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true, dep_done = false;
            int it = 0;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
                const int m = tile / args.n_tiles, n = tile % args.n_tiles;
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, args.status);
                    if (!ok) break;
                    mbar_expect_tx(full_bar(stage), S::STAGE_BYTES);
                    const uint32_t sa = base + stage * S::STAGE_BYTES;
                    tma_load_2d(sa, &tm_x, kb * BK, m * BM, full_bar(stage));
                    tma_load_2d(sa + S::A_BYTES, &tm_w, kb * BK, n * BN, full_bar(stage));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                const int ns = tile_ns(it, m);
                if (ns > 0 && !dep_done) { dep_wait(); dep_done = true; }     // t comes from the shrink kernel
                for (int g0 = 0; g0 < ns && ok; g0 += SLABS_PER_STAGE) {
                    const int cnt = min(SLABS_PER_STAGE, ns - g0);
                    ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, args.status);
                    if (!ok) break;
                    mbar_expect_tx(full_bar(stage), cnt * (S::T_SLAB_BYTES + S::B_SLAB_BYTES));
                    const uint32_t sa = base + stage * S::STAGE_BYTES;
                    for (int i = 0; i < cnt; ++i) {
                        const int slot = m * args.slab_cap + g0 + i;
                        const int slab = tile_slab_id(it, m, g0 + i);
                        tma_load_2d(sa + i * S::T_SLAB_BYTES, &tm_t, 0, slot * BM, full_bar(stage));
                        tma_load_2d(sa + S::A_BYTES + i * S::B_SLAB_BYTES, &tm_bt, 0,
                                    slab * args.n_out + n * BN, full_bar(stage));
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = instr_desc(BN);
            // Descriptors of stage 0; a stage adds STAGE_BYTES / 16 and a K step of 16 adds 2 to the
            // address field.  Keeping the issuing thread's work per K block to a handful of
            // instructions matters: the tensor pipe runs dry whenever this thread is late.
            const uint64_t da0 = smem_desc(base, 128), db0 = smem_desc(base + S::A_BYTES, 128);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
                const int m = tile / args.n_tiles;
                const int ns = tile_ns(it, m);
                ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, args.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                uint32_t accumulate = 0;
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    ok = mbar_wait(full_bar(stage), phase, abort_flag, args.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t so = (uint64_t)(stage * (S::STAGE_BYTES >> 4));
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        umma_bf16(d_tmem, da0 + so + 2 * k, db0 + so + 2 * k, idesc, accumulate);
                        accumulate = 1;
                    }
                    umma_commit(empty_bar(stage));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                for (int g0 = 0; g0 < ns && ok; g0 += SLABS_PER_STAGE) {
                    const int cnt = min(SLABS_PER_STAGE, ns - g0);
                    ok = mbar_wait(full_bar(stage), phase, abort_flag, args.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = base + stage * S::STAGE_BYTES;
                    const uint32_t sb = sa + S::A_BYTES;
                    for (int i = 0; i < cnt; ++i) {
                        umma_bf16(d_tmem, smem_desc(sa + i * S::T_SLAB_BYTES, 32),
                                  smem_desc(sb + i * S::B_SLAB_BYTES, 32), idesc, accumulate);
                        accumulate = 1;
                    }
                    umma_commit(empty_bar(stage));
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(tfull_bar(acc));
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..)
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31
        const int half = (warp - 2) >> 2;             // which share of the tile's 32-column chunks
        const uint32_t staging = base + S::STAGING_OFFSET + (uint32_t)(warp - 2) * STAGING_BYTES_PER_WARP;
        dep_wait();                                   // the row statistics come from the shrink kernel
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t chunk_no = 0;                        // running chunk counter: picks the staging buffer
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
            const int m = tile / args.n_tiles, n = tile % args.n_tiles;
            ok = epilogue_tile<BN, EPI, HALVES, false, LNF, false>(args, tm_y, staging, chunk_no, tmem_base, acc,
                                                              acc_phase, tfull_bar(acc), tempty_bar(acc), abort_flag,
                                                              m, n, quarter, half, lane, nullptr, 0u, 0u, 0u);
            if (!ok) break;
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (args.tma_store && lane == 0) bulk_wait_all();
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    dep_wait();               // never finish before the kernel this one was allowed to overtake
    if (*abort_flag) {
        // give copies and MMAs still in flight time to land before shared memory / TMEM go away
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * BN);
    }
}

// ---------------------------------------------------------------------------------------
// The same GEMM on CTA pairs (n_out a multiple of 256).  Two CTAs of a cluster share one
// 256 x 256 output tile: each stages its own 128 rows of x (and of the t slabs) and HALF of the
// W^T tile (and of the B slabs), so every byte of W^T crosses the L2 -> SM fabric once per 256
// rows instead of once per 128, and one tcgen05.mma.cta_group::2 (M = 256) issued by the even
// CTA drives the tensor cores of both SMs, each accumulating its own 128 rows in its own TMEM.
//   full[s]    (even CTA)   bytes of both CTAs' loads of stage s (the odd CTA's TMA signals it)
//   empty[s]   (both CTAs)  the pair MMAs that read stage s are done (multicast commit)
//   tfull[a]   (both CTAs)  accumulator a is complete (multicast commit)
//   tempty[a]  (even CTA)   both CTAs' epilogue warps have drained accumulator a
// Six 32 KB stages per CTA.  No TMA multicast is used.
// ---------------------------------------------------------------------------------------
constexpr int P_BN = 256;
constexpr int P_EW = 8;
// Ring depth and residual landing area by epilogue: the residual epilogue trades two of the six 32 KB
// stages for a 64 KB area into which TMA fetches the tile's residual rows ahead of the accumulator.
template <int EPI, bool RESS>
struct PairCfg {
    static constexpr bool RES = EPI == EPI_RESIDUAL && RESS;
    static constexpr int STAGES = RES ? 4 : 6;
    static constexpr int RES_BYTES_PER_WARP = RES ? 4 * 32 * 64 : 0;       // four [32 rows x 32 bf16] chunks
};
constexpr int P_A_BYTES = BM * BK * 2;                 // 16 KB: this CTA's 128 rows of x
constexpr int P_B_BYTES = (P_BN / 2) * BK * 2;         // 16 KB: this CTA's half of the W^T tile
constexpr int P_STAGE_BYTES = P_A_BYTES + P_B_BYTES;
constexpr int P_T_SLAB_BYTES = BM * PM_SLAB * 2;       // 4 KB
constexpr int P_B_SLAB_BYTES = (P_BN / 2) * PM_SLAB * 2;   // 4 KB
constexpr int P_MAX_STAGES = 6;
constexpr int P_STAGING_OFFSET = P_MAX_STAGES * P_STAGE_BYTES;      // stages, then (residual kernels) the
constexpr int P_PLAN_OFFSET = P_STAGING_OFFSET + P_EW * STAGING_BYTES_PER_WARP;   // residual area inside them
constexpr int P_BAR_OFFSET = P_PLAN_OFFSET + PLAN_BYTES;
constexpr int P_SMEM_TOTAL = P_BAR_OFFSET + 256;
constexpr int P_THREADS = 64 + 32 * P_EW;

// RESS (residual epilogue only): residual through shared memory with a four-stage ring (short K, where
// the epilogue is exposed) instead of per-thread loads with the full six stages (long K).
template <int EPI, bool LNF, bool RESS>
__global__ void __launch_bounds__(P_THREADS, 1)
lora_gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                      const __grid_constant__ CUtensorMap tm_t, const __grid_constant__ CUtensorMap tm_bt,
                      const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_res,
                      const GemmArgs args) {
    constexpr int BN = P_BN;
    constexpr int HALVES = P_EW / 4;
    constexpr int P_STAGES = PairCfg<EPI, RESS>::STAGES;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    const uint32_t rank = cluster_ctarank();          // 0: issues the MMAs, 1: its peer
    uint8_t* smem = smem_raw;
    const uint32_t bars = base + P_BAR_OFFSET;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (P_MAX_STAGES + s); };
    auto tfull_bar = [&](int s) { return bars + 8u * (2 * P_MAX_STAGES + s); };
    auto tempty_bar = [&](int s) { return bars + 8u * (2 * P_MAX_STAGES + 2 + s); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + P_BAR_OFFSET + 8 * (2 * P_MAX_STAGES + 4));
    // the peer CTA's TMEM base: written only by the peer (any time before the cluster barrier below),
    // never by this CTA, so there is no ordering to get wrong
    volatile uint32_t* peer_slot = tmem_slot + 1;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + P_BAR_OFFSET + 8 * (2 * P_MAX_STAGES + 4) + 8);
    // res_bar[w]: the residual rows of epilogue warp w's chunks have landed (residual kernels)
    auto res_bar = [&](int w) { return bars + 8u * (2 * P_MAX_STAGES + 4) + 24u + 8u * w; };
    int* plan = reinterpret_cast<int*>(smem + P_PLAN_OFFSET);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int total_tiles = args.m_tiles * args.n_tiles;      // m_tiles counts 256-row tiles here
    const int num_kb = args.k_in / BK;

    // LoRA plan of this CTA's tiles (both halves of a 256-row tile carry the same slab list)
    const int plan_stride = 1 + args.slab_cap;
    const int plan_tiles = args.tile_nslabs ? PLAN_BYTES / (4 * plan_stride) : 0;
    if (args.tile_nslabs) {
        for (int i = threadIdx.x / 8; i < plan_tiles; i += P_THREADS / 8) {
            const int tile = pair_id + i * n_pairs;
            if (tile >= total_tiles) break;
            const int m = 2 * (tile / args.n_tiles) + (int)rank;
            const int ns = args.tile_nslabs[m];
            if ((threadIdx.x & 7) == 0) plan[i * plan_stride] = ns;
            for (int q = threadIdx.x & 7; q < ns; q += 8) plan[i * plan_stride + 1 + q] = args.tile_slab[m * args.slab_cap + q];
        }
    }
    auto tile_ns = [&](int it, int m) -> int {
        if (!args.tile_nslabs) return 0;
        return it < plan_tiles ? plan[it * plan_stride] : args.tile_nslabs[m];
    };
    auto tile_slab_id = [&](int it, int m, int q) -> int {
        return it < plan_tiles ? plan[it * plan_stride + 1 + q] : args.tile_slab[m * args.slab_cap + q];
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(tfull_bar(s), 1); mbar_init(tempty_bar(s), 2 * P_EW); }
        for (int w = 0; w < P_EW; ++w) mbar_init(res_bar(w), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32((const void*)tmem_slot), 512);     // all of this SM's tensor memory
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // both CTAs must hold the same TMEM columns (the pair MMA uses one address for both); tell the peer
    if (threadIdx.x == 0) st_cluster_u32(mapa_cluster(smem_u32((const void*)peer_slot), rank ^ 1u), tmem_base);
    cluster_sync_all();          // barriers initialised and TMEM bases exchanged in both CTAs
    const bool usable = ((base & 1023u) == 0) && (*peer_slot == tmem_base);
    if (!usable && threadIdx.x == 0) atomicCAS(args.status, 0, (int)PM_ERR_CUDA);

    if (!usable) {
        // fall through to the teardown
    } else if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true, dep_done = false;
            int it = 0;
            for (int tile = pair_id; tile < total_tiles && ok; tile += n_pairs, ++it) {
                const int m2 = tile / args.n_tiles, n = tile % args.n_tiles;
                const int m = 2 * m2 + (int)rank;                   // this CTA's 128-row tile
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    ok = mbar_wait_cluster(empty_bar(stage), phase ^ 1u, abort_flag, args.status);
                    if (!ok) break;
                    const uint32_t fb = mapa_cluster(full_bar(stage), 0);
                    if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * P_STAGE_BYTES);
                    const uint32_t sa = base + stage * P_STAGE_BYTES;
                    tma_load_2d_pair(sa, &tm_x, kb * BK, m * BM, fb);
                    tma_load_2d_pair(sa + P_A_BYTES, &tm_w, kb * BK, n * BN + (int)rank * (BN / 2), fb);
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
                const int ns = tile_ns(it, m);
                if (ns > 0 && !dep_done) { dep_wait(); dep_done = true; }     // t comes from the shrink kernel
                for (int g0 = 0; g0 < ns && ok; g0 += SLABS_PER_STAGE) {
                    const int cnt = min(SLABS_PER_STAGE, ns - g0);
                    ok = mbar_wait_cluster(empty_bar(stage), phase ^ 1u, abort_flag, args.status);
                    if (!ok) break;
                    const uint32_t fb = mapa_cluster(full_bar(stage), 0);
                    if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * cnt * (P_T_SLAB_BYTES + P_B_SLAB_BYTES));
                    const uint32_t sa = base + stage * P_STAGE_BYTES;
                    for (int i = 0; i < cnt; ++i) {
                        const int slot = m * args.slab_cap + g0 + i;
                        const int slab = tile_slab_id(it, m, g0 + i);
                        tma_load_2d_pair(sa + i * P_T_SLAB_BYTES, &tm_t, 0, slot * BM, fb);
                        tma_load_2d_pair(sa + P_A_BYTES + i * P_B_SLAB_BYTES, &tm_bt, 0,
                                         slab * args.n_out + n * BN + (int)rank * (BN / 2), fb);
                    }
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_pair(BN);
            const uint64_t da0 = smem_desc(base, 128), db0 = smem_desc(base + P_A_BYTES, 128);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            int it = 0;
            for (int tile = pair_id; tile < total_tiles && ok; tile += n_pairs, ++it) {
                const int m = 2 * (tile / args.n_tiles);
                const int ns = tile_ns(it, m);
                ok = mbar_wait_cluster(tempty_bar(acc), acc_phase ^ 1u, abort_flag, args.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                uint32_t accumulate = 0;
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    ok = mbar_wait_cluster(full_bar(stage), phase, abort_flag, args.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t so = (uint64_t)(stage * (P_STAGE_BYTES >> 4));
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        umma_bf16_pair(d_tmem, da0 + so + 2 * k, db0 + so + 2 * k, idesc, accumulate);
                        accumulate = 1;
                    }
                    umma_commit_pair(empty_bar(stage));
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
                for (int g0 = 0; g0 < ns && ok; g0 += SLABS_PER_STAGE) {
                    const int cnt = min(SLABS_PER_STAGE, ns - g0);
                    ok = mbar_wait_cluster(full_bar(stage), phase, abort_flag, args.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = base + stage * P_STAGE_BYTES;
                    const uint32_t sb = sa + P_A_BYTES;
                    for (int i = 0; i < cnt; ++i) {
                        umma_bf16_pair(d_tmem, smem_desc(sa + i * P_T_SLAB_BYTES, 32),
                                       smem_desc(sb + i * P_B_SLAB_BYTES, 32), idesc, accumulate);
                        accumulate = 1;
                    }
                    umma_commit_pair(empty_bar(stage));
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit_pair(tfull_bar(acc));
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs)
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        const uint32_t staging = base + P_STAGING_OFFSET + (uint32_t)(warp - 2) * STAGING_BYTES_PER_WARP;
        dep_wait();                                   // the row statistics come from the shrink kernel
        int acc = 0;
        uint32_t acc_phase = 0, res_phase = 0;
        uint32_t chunk_no = 0;
        bool ok = true;
        for (int tile = pair_id; tile < total_tiles && ok; tile += n_pairs) {
            const int m = 2 * (tile / args.n_tiles) + (int)rank, n = tile % args.n_tiles;
            ok = epilogue_tile<BN, EPI, HALVES, true, LNF, PairCfg<EPI, RESS>::RES>(
                args, tm_y, staging, chunk_no, tmem_base, acc, acc_phase, tfull_bar(acc),
                mapa_cluster(tempty_bar(acc), 0), abort_flag, m, n, quarter, half, lane, &tm_res,
                base + PairCfg<EPI, RESS>::STAGES * P_STAGE_BYTES + (uint32_t)(warp - 2) * PairCfg<EPI, RESS>::RES_BYTES_PER_WARP,
                res_bar(warp - 2), res_phase);
            res_phase ^= 1u;
            if (!ok) break;
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (args.tma_store && lane == 0) bulk_wait_all();
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    dep_wait();               // never finish before the kernel this one was allowed to overtake
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);    // let copies / MMAs in flight land
    }
    tc_fence_before();
    cluster_sync_all();          // the peer no longer reads this CTA's shared memory or signals its barriers
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ---------------------------------------------------------------------------------------
// shrink on the tensor cores: t[tile][s][row][j] = mask(row) * s_a * sum_k x[row,k] A_a[k, 16 s' + j]
//
// One CTA per 128-row tile, three CTAs per SM, so every tile of a batch is in flight at once and the
// kernel runs at the speed of its one pass over x (a persistent walk of a few tiles per CTA spent
// most of a launch ramping up and waiting for the CTAs that drew one tile more).  Inside a tile the
// LoRA slabs are taken in groups of up to eight: per group the x tile streams through shared memory
// once (TMA, 128B swizzle) next to the group's A^T slabs (16 arena rows per slab, stacked), one UMMA
// of N = 16 * slabs per 16 K-columns accumulates in tensor memory, and the epilogue warps scale,
// mask, round to bf16 and store each slab as a [128 x 16] block -- the layout the fused GEMM fetches
// as a 32B-swizzled operand.  The ring's stage size follows the tile's own slab count, so a tile with
// few slabs gets more stages out of the same shared memory.
// ---------------------------------------------------------------------------------------
struct ShrinkArgs {
    int rows, k_in, slab_cap, n_tiles;
    int reverse;                   // visit the tiles from the last row tile down (see launch_shrink)
    const int* tile_nslabs;
    const int* tile_slab;
    const float* tile_scale;
    const uint32_t* tile_mask;
    bf16* tbuf;
    int* status;
    // LayerNorm folded into the adapters (x is the raw residual stream, the arena holds gamma o A):
    //   t = s (rstd (x A' - mean c1) + c2);  stored divided by rstd, because the fused GEMM applies
    //   rstd to its whole accumulator, base and LoRA part alike
    const float2* ln_stats;     // null = not folded, or the statistics are computed here (stats_out)
    const float* ln_c1;
    const float* ln_c2;
    // Statistics mode: the epilogue warps also read every x block as it passes through shared memory
    // and produce each row's (mean, 1/sqrt(var + eps)) -- used for t right away and written to
    // stats_out for the GEMM that follows.  Every row tile is then visited, with or without slabs.
    float2* stats_out;
    float ln_eps;
    int ring_bytes, max_stages;       // the stage ring of a CTA
};

constexpr int SHRINK_MAX_STAGES = 8;
constexpr int SHRINK_GROUP = 8;                       // slabs per pass over x: 128 accumulator columns
constexpr int SHRINK_X_BYTES = BM * BK * 2;           // 16 KB
constexpr int SHRINK_A_SLAB_BYTES = PM_SLAB * BK * 2; // 2 KB: 16 arena rows x 64 K-columns
// The ring of x / slab stages.  Full grids (three CTAs per SM): 72 KB, at most four stages -- 4 stages with one
// slab, 3 up to four, 2 up to eight.  Grids of no more CTAs than SMs (a few frames): a CTA has its SM to
// itself and nothing else hides the latency of its loads, so it takes 192 KB and up to eight stages.
constexpr int SHRINK_RING_BYTES = 72 * 1024;
constexpr int SHRINK_RING_BYTES_ALONE = 192 * 1024;
constexpr int SHRINK_SMEM_MAX = SHRINK_RING_BYTES_ALONE + 256;

__global__ void __launch_bounds__(SHRINK_THREADS)
shrink_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_at,
                 const ShrinkArgs args) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = smem_u32(smem);
    if (base & 1023u) {                       // swizzled operands need a 1024-byte aligned window
        if (threadIdx.x == 0) atomicCAS(args.status, 0, (int)PM_ERR_CUDA);
        return;
    }
    const int tile = args.reverse ? args.n_tiles - 1 - (int)blockIdx.x : (int)blockIdx.x;
    const int ns = args.tile_nslabs[tile];
    const bool stats = args.stats_out != nullptr;
    if (ns == 0 && !stats) return;            // nothing to do for this tile (the whole CTA leaves; an exited CTA
                                              // counts as having released the kernel's dependents)
    const int sg = min(ns, SHRINK_GROUP);
    const int stage_bytes = SHRINK_X_BYTES + sg * SHRINK_A_SLAB_BYTES;
    const int STG = min(args.max_stages, args.ring_bytes / stage_bytes);
    // groups of slabs; in statistics mode a tile without slabs still makes one pass over x
    const int n_groups = ns == 0 ? 1 : (ns + SHRINK_GROUP - 1) / SHRINK_GROUP;
    uint32_t acc_cols = 32;                   // power of two >= 16 * sg
    while ((int)acc_cols < sg * PM_SLAB) acc_cols <<= 1;

    const uint32_t bars = base + (uint32_t)args.ring_bytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (SHRINK_MAX_STAGES + s); };
    const uint32_t tfull_bar = bars + 8u * (2 * SHRINK_MAX_STAGES);
    const uint32_t tempty_bar = bars + 8u * (2 * SHRINK_MAX_STAGES + 1);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + args.ring_bytes + 8 * (2 * SHRINK_MAX_STAGES + 2));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + args.ring_bytes + 8 * (2 * SHRINK_MAX_STAGES + 2) + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = args.k_in / BK;

    if (threadIdx.x == 0) {
        // a stage is free again when its MMAs are done and, in statistics mode, the four epilogue warps
        // have read it too
        for (int s = 0; s < STG; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), stats ? 5 : 1); }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1 && ns > 0) {
        tmem_alloc(smem_u32((const void*)tmem_slot), acc_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ns > 0 ? *tmem_slot : 0u;
    // The fused GEMM that follows needs t (and the row statistics) only when its first tile's base K loop
    // is over: it may start on every SM this kernel's CTAs have left, while the slowest tiles finish.
    dep_release();

    if (warp == 0) {
        if (lane == 0) {
            // -------------------------------------------------------------- TMA producer
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int g = 0; g < n_groups && ok; ++g) {
                const int g0 = g * SHRINK_GROUP;
                const int cnt = max(0, min(SHRINK_GROUP, ns - g0));
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, args.status);
                    if (!ok) break;
                    mbar_expect_tx(full_bar(stage), SHRINK_X_BYTES + cnt * SHRINK_A_SLAB_BYTES);
                    const uint32_t sa = base + stage * stage_bytes;
                    tma_load_2d(sa, &tm_x, kb * BK, tile * BM, full_bar(stage));
                    for (int i = 0; i < cnt; ++i) {
                        const int slab = args.tile_slab[tile * args.slab_cap + g0 + i];
                        tma_load_2d(sa + SHRINK_X_BYTES + i * SHRINK_A_SLAB_BYTES, &tm_at, kb * BK,
                                    slab * PM_SLAB, full_bar(stage));
                    }
                    if (++stage == STG) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // -------------------------------------------------------------- MMA issuer
            const uint64_t da0 = smem_desc(base, 128), db0 = smem_desc(base + SHRINK_X_BYTES, 128);
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int g = 0; g < n_groups && ok; ++g) {
                const int g0 = g * SHRINK_GROUP;
                const int cnt = max(0, min(SHRINK_GROUP, ns - g0));
                if (cnt == 0) {            // statistics only: hand the stages straight back
                    for (int kb = 0; kb < num_kb && ok; ++kb) {
                        ok = mbar_wait(full_bar(stage), phase, abort_flag, args.status);
                        if (!ok) break;
                        mbar_arrive(empty_bar(stage));
                        if (++stage == STG) { stage = 0; phase ^= 1u; }
                    }
                    continue;
                }
                const uint32_t idesc = instr_desc(cnt * PM_SLAB);
                // the one accumulator: the epilogue warps have drained the previous group
                ok = mbar_wait(tempty_bar, acc_phase ^ 1u, abort_flag, args.status);
                if (!ok) break;
                tc_fence_after();
                uint32_t accumulate = 0;
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    ok = mbar_wait(full_bar(stage), phase, abort_flag, args.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t so = (uint64_t)((stage * stage_bytes) >> 4);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        umma_bf16(tmem_base, da0 + so + 2 * k, db0 + so + 2 * k, idesc, accumulate);
                        accumulate = 1;
                    }
                    umma_commit(empty_bar(stage));
                    if (++stage == STG) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(tfull_bar);
                acc_phase ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;
        int stage = 0;
        uint32_t acc_phase = 0, phase = 0;
        bool ok = true;
        float mean = 0.f, inv_rstd = 0.f;
        for (int g = 0; g < n_groups && ok; ++g) {
            const int g0 = g * SHRINK_GROUP;
            const int cnt = max(0, min(SHRINK_GROUP, ns - g0));
            if (stats) {
                // follow the ring: on the tile's first pass every thread sums its row of each x block,
                // shifted by the row's first element (which keeps the sum of squares well conditioned);
                // the arithmetic runs on pairs (packed fp32): the two halves are added at the end
                float pivot = 0.f;
                uint64_t npivot2 = 0, s1p = pk2(0.f, 0.f), s2p = pk2(0.f, 0.f);
                for (int kb = 0; kb < num_kb && ok; ++kb) {
                    ok = mbar_wait(full_bar(stage), phase, abort_flag, args.status);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    if (g == 0) {
                        const uint32_t row_addr = base + stage * stage_bytes + r * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            uint4 q;
                            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(q.x), "=r"(q.y), "=r"(q.z), "=r"(q.w)
                                         : "r"(row_addr + ((c ^ (r & 7)) << 4)));
                            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
                            if (kb == 0 && c == 0) {
                                pivot = __uint_as_float(w[0] << 16);
                                npivot2 = pk2(-pivot, -pivot);
                            }
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const uint64_t a = add2(pk2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xFFFF0000u)), npivot2);
                                s1p = add2(s1p, a);
                                s2p = fma2(a, a, s2p);
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_bar(stage));
                    if (++stage == STG) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (g == 0) {
                    float s1a, s1b, s2a, s2b;
                    upk2(s1p, s1a, s1b);
                    upk2(s2p, s2a, s2b);
                    const float inv_d = 1.f / (float)args.k_in;
                    const float m1 = (s1a + s1b) * inv_d;
                    const float var = fmaxf((s2a + s2b) * inv_d - m1 * m1, 0.f);
                    const float rstd = rsqrtf(var + args.ln_eps);
                    mean = pivot + m1;
                    inv_rstd = 1.f / rstd;
                    if (tile * BM + r < args.rows) args.stats_out[tile * BM + r] = make_float2(mean, rstd);
                }
                if (cnt == 0) continue;
            }
            ok = mbar_wait(tfull_bar, acc_phase, abort_flag, args.status);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
            if (args.ln_stats && tile * BM + r < args.rows) {
                const float2 st = args.ln_stats[tile * BM + r];
                mean = st.x;
                inv_rstd = 1.f / st.y;
            }
            for (int i = 0; i < cnt; ++i) {
                const int slot = tile * args.slab_cap + g0 + i;
                uint32_t v[16];
                tmem_ld16(t_row + (uint32_t)(i * PM_SLAB), v);
                tmem_ld_wait();
                const bool on = (args.tile_mask[(size_t)slot * 4 + quarter] >> lane) & 1u;
                const float sc = on ? args.tile_scale[slot] : 0.f;
                if (args.ln_stats || stats) {
                    const float* c1 = args.ln_c1 + (size_t)args.tile_slab[slot] * PM_SLAB;
                    const float* c2 = args.ln_c2 + (size_t)args.tile_slab[slot] * PM_SLAB;
#pragma unroll
                    for (int j = 0; j < PM_SLAB; ++j)
                        v[j] = __float_as_uint(fmaf(-mean, __ldg(c1 + j), __uint_as_float(v[j])) +
                                               inv_rstd * __ldg(c2 + j));
                }
                uint4 o[2];
                uint32_t* ow = reinterpret_cast<uint32_t*>(o);
#pragma unroll
                for (int j = 0; j < PM_SLAB; j += 2)
                    ow[j >> 1] = pack_bf16(__uint_as_float(v[j]) * sc, __uint_as_float(v[j + 1]) * sc);
                uint4* dst = reinterpret_cast<uint4*>(args.tbuf + ((size_t)slot * BM + r) * PM_SLAB);
                dst[0] = o[0];
                dst[1] = o[1];
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar);
            acc_phase ^= 1u;
        }
    }
    __syncwarp();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1 && ns > 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, acc_cols);
    }
}

// Exercises the give-up path of the bounded waits without any fault: one CTA with the warp roles of
// the kernels above allocates tensor memory, then its "MMA" thread waits -- with the caller's cycle
// limit -- on an mbarrier nothing ever arrives on.  The wait must expire, raise the abort flag and
// record PM_ERR_TIMEOUT; the other warps, parked on a second barrier, must see the abort flag and
// leave too; the CTA drains, frees its tensor memory and returns.  trace[0] = the timed-out wait
// returned false, trace[1] = warps that left through the abort flag, trace[2] = 1 after the release.
__global__ void __launch_bounds__(128) wait_timeout_selftest_kernel(long long limit, int* status, int* trace) {
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), 32);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    if (warp == 1) {
        if (lane == 0) {
            const bool ok = mbar_wait(smem_u32(&bars[0]), 0u, abort_flag, status, limit);
            trace[0] = ok ? 0 : 1;
        }
    } else {
        // like an epilogue warp waiting for an accumulator that never comes: ends through the abort flag
        bool ok = mbar_wait(smem_u32(&bars[1]), 0u, abort_flag, status);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok && lane == 0) atomicAdd(&trace[1], 1);
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 32);
        if (lane == 0) trace[2] = 1;
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

CUtensorMapSwizzle swz(int bytes) {
    return bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
         : bytes == 64  ? CU_TENSOR_MAP_SWIZZLE_64B
         : bytes == 32  ? CU_TENSOR_MAP_SWIZZLE_32B
                        : CU_TENSOR_MAP_SWIZZLE_NONE;
}

}  // namespace

extern "C" int pm_selftest_wait_timeout(long long limit_cycles, int32_t* status, int32_t* trace, void* cuda_stream) {
    // the other warps' own limit is the library's (~2 s): the test limit must stay far below it
    if (!status || !trace || limit_cycles <= 0 || limit_cycles > 100000000ll) return PM_ERR_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(trace, 0, 3 * sizeof(int32_t), st) != cudaSuccess) return PM_ERR_CUDA;
    wait_timeout_selftest_kernel<<<1, 128, 0, st>>>(limit_cycles, status, trace);
    return cudaGetLastError() == cudaSuccess ? PM_OK : PM_ERR_CUDA;
}

bool tm_encode_2d(CUtensorMap* tm, const void* base, uint64_t inner, uint64_t outer,
                  uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, int swizzle) {
    EncodeTiledFn fn = get_encode();
    if (!fn) return false;
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {row_stride_bytes};
    const cuuint32_t box[2] = {box_inner, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swz(swizzle), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tm_encode_3d(CUtensorMap* tm, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                  uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1,
                  uint32_t b2, int swizzle) {
    EncodeTiledFn fn = get_encode();
    if (!fn) return false;
    const cuuint64_t dims[3] = {d0, d1, d2};
    const cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
    const cuuint32_t box[3] = {b0, b1, b2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swz(swizzle), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_shrink(const Launch& L, const LinearDev& lin, const RouteDev& R,
                          const CUtensorMap* tm_x, const bf16* /*x*/, int rows, bf16* tbuf, int n_sms,
                          const float2* ln_stats, float2* stats_out, float ln_eps) {
    if (R.n_tiles <= 0) return cudaSuccess;
    if (R.slab_cap <= 0) return stats_out ? cudaErrorInvalidValue : cudaSuccess;   // nothing to shrink
    ShrinkArgs a;
    a.rows = rows; a.k_in = lin.k_in; a.slab_cap = R.slab_cap; a.n_tiles = R.n_tiles;
    a.tile_nslabs = R.tile_nslabs; a.tile_slab = R.tile_slab; a.tile_scale = R.tile_scale;
    a.tile_mask = R.tile_mask; a.tbuf = tbuf; a.status = L.status;
    // a linear with LayerNorm folded in gets the row statistics either ready-made or computed here
    if ((lin.ln_g != nullptr) != ((ln_stats != nullptr) != (stats_out != nullptr))) return cudaErrorInvalidValue;
    a.ln_stats = ln_stats; a.ln_c1 = lin.ln_c1; a.ln_c2 = lin.ln_c2;
    a.stats_out = stats_out; a.ln_eps = ln_eps;
    // x larger than the L2 cache was written front to back by the kernel before this one, so its tail
    // is what the cache still holds: start there, and leave the front in the cache for the GEMM that
    // follows (which walks front to back)
    a.reverse = (size_t)rows * lin.k_in * sizeof(bf16) > ((size_t)96 << 20) ? 1 : 0;
    static SmemGrant grant;
    if (cudaError_t e = grant.ensure(shrink_tc_kernel, SHRINK_SMEM_MAX); e != cudaSuccess) return e;
    const bool alone = n_sms > 0 && a.n_tiles <= n_sms;
    a.ring_bytes = alone ? SHRINK_RING_BYTES_ALONE : SHRINK_RING_BYTES;
    a.max_stages = alone ? SHRINK_MAX_STAGES : 4;
    ProfScope ps(L, KC_SHRINK);
    shrink_tc_kernel<<<a.n_tiles, SHRINK_THREADS, a.ring_bytes + 256, L.st>>>(*tm_x, lin.tm_at, a);
    BUMP(L);
    return cudaGetLastError();
}

#ifndef PM_GEMM_EPI_WARPS
#define PM_GEMM_EPI_WARPS 8
#endif
constexpr int GEMM_EPI_WARPS = PM_GEMM_EPI_WARPS;      // 4 or 8

template <int BN, int EPI, bool LNF = false>
static cudaError_t launch_gemm_bn(const Launch& L, const CUtensorMap& tm_x, const CUtensorMap& tm_w,
                                  const CUtensorMap& tm_t, const CUtensorMap& tm_bt, const CUtensorMap& tm_y,
                                  const GemmArgs& a, int n_sms) {
    constexpr int EW = GEMM_EPI_WARPS;
    static SmemGrant grant;
    if (cudaError_t e = grant.ensure(lora_gemm_kernel<BN, EPI, EW, LNF>, Smem<BN, EW>::TOTAL); e != cudaSuccess) return e;
    const int total = a.m_tiles * a.n_tiles;
    const int grid = total < n_sms ? total : n_sms;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(64 + 32 * EW);
    cfg.dynamicSmemBytes = Smem<BN, EW>::TOTAL;
    cfg.stream = L.st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.overlap_prev ? 1 : 0;
    ProfScope ps(L, KC_GEMM);
    cudaError_t e = cudaLaunchKernelEx(&cfg, lora_gemm_kernel<BN, EPI, EW, LNF>, tm_x, tm_w, tm_t, tm_bt, tm_y, a);
    BUMP(L);
    return e != cudaSuccess ? e : cudaGetLastError();
}

template <int BN>
static cudaError_t launch_gemm_epi(const Launch& L, const CUtensorMap& tm_x, const CUtensorMap& tm_w,
                                   const CUtensorMap& tm_t, const CUtensorMap& tm_bt, const CUtensorMap& tm_y,
                                   const GemmArgs& a, int n_sms) {
    if (a.ln_stats) {        // LayerNorm folded in: only the epilogues that follow a LayerNorm
        if (a.epi == EPI_GELU) return launch_gemm_bn<BN, EPI_GELU, true>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        if (a.epi == EPI_NONE) return launch_gemm_bn<BN, EPI_NONE, true>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        return cudaErrorInvalidValue;
    }
    switch (a.epi) {
        case EPI_GELU: return launch_gemm_bn<BN, EPI_GELU>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        case EPI_RESIDUAL: return launch_gemm_bn<BN, EPI_RESIDUAL>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        case EPI_PATCH: return launch_gemm_bn<BN, EPI_PATCH>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        default: return launch_gemm_bn<BN, EPI_NONE>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
    }
}

template <int EPI, bool LNF = false, bool RESS = false>
static cudaError_t launch_gemm_pair(const Launch& L, const CUtensorMap& tm_x, const CUtensorMap& tm_w,
                                    const CUtensorMap& tm_t, const CUtensorMap& tm_bt, const CUtensorMap& tm_y,
                                    const GemmArgs& a, int n_sms) {
    // the residual tile is fetched by TMA with the output's geometry (32 x 32 boxes, 64B swizzle)
    CUtensorMap tm_res = tm_y;
    if (EPI == EPI_RESIDUAL && (const void*)a.residual != (const void*)a.y) {
        if (!tm_encode_2d(&tm_res, a.residual, a.n_out, a.rows, (uint64_t)a.n_out * 2, 32, 32, 64))
            return cudaErrorInvalidValue;
    }
    static SmemGrant grant;
    if (cudaError_t e = grant.ensure(lora_gemm_pair_kernel<EPI, LNF, RESS>, P_SMEM_TOTAL); e != cudaSuccess) return e;
    const int total = a.m_tiles * a.n_tiles;
    const int pairs = total < n_sms / 2 ? total : n_sms / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(P_THREADS);
    cfg.dynamicSmemBytes = P_SMEM_TOTAL;
    cfg.stream = L.st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.overlap_prev ? 2 : 1;
    ProfScope ps(L, KC_GEMM);
    cudaError_t e = cudaLaunchKernelEx(&cfg, lora_gemm_pair_kernel<EPI, LNF, RESS>, tm_x, tm_w, tm_t, tm_bt, tm_y, tm_res, a);
    BUMP(L);
    return e != cudaSuccess ? e : cudaGetLastError();
}

static cudaError_t launch_gemm_pair_epi(const Launch& L, const CUtensorMap& tm_x, const CUtensorMap& tm_w,
                                        const CUtensorMap& tm_t, const CUtensorMap& tm_bt, const CUtensorMap& tm_y,
                                        const GemmArgs& a, int n_sms) {
    if (a.ln_stats) {
        if (a.epi == EPI_GELU) return launch_gemm_pair<EPI_GELU, true>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        if (a.epi == EPI_NONE) return launch_gemm_pair<EPI_NONE, true>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        return cudaErrorInvalidValue;
    }
    switch (a.epi) {
        case EPI_GELU: return launch_gemm_pair<EPI_GELU>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        case EPI_RESIDUAL:
            if (a.k_in <= 1024) return launch_gemm_pair<EPI_RESIDUAL, false, true>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
            return launch_gemm_pair<EPI_RESIDUAL>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        case EPI_PATCH: return launch_gemm_pair<EPI_PATCH>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
        default: return launch_gemm_pair<EPI_NONE>(L, tm_x, tm_w, tm_t, tm_bt, tm_y, a, n_sms);
    }
}

// lin.tm_w / lin.tm_bt are encoded for the BN chosen by gemm_tile_n(lin.n_out); lin.tm_w_half /
// lin.tm_bt_half (n_out a multiple of 256) fetch 128 of a tile's 256 columns for the pair kernel.
int gemm_tile_n(int n_out) { return (n_out % 256 == 0) ? 256 : 128; }

cudaError_t launch_lora_gemm(const Launch& L, const LinearDev& lin, const RouteDev* R,
                             const CUtensorMap& tm_x, const CUtensorMap* tm_t, const CUtensorMap* tm_y,
                             int rows, int epi, const bf16* residual, const PatchEpi& pe, bf16* y,
                             int n_sms, const float2* ln_stats, bool after_shrink) {
    if (rows <= 0) return cudaSuccess;
    if ((lin.ln_g != nullptr) != (ln_stats != nullptr)) return cudaErrorInvalidValue;
    const int bn = gemm_tile_n(lin.n_out);
    GemmArgs a;
    a.rows = rows; a.k_in = lin.k_in; a.n_out = lin.n_out;
    a.m_tiles = (rows + BM - 1) / BM;
    a.n_tiles = (lin.n_out + bn - 1) / bn;
    a.epi = epi; a.bias = lin.bias; a.residual = residual; a.y = y; a.pe = pe;
    const bool lora = R && tm_t && R->slab_cap > 0 && lin.lora.At != nullptr;
    a.tile_nslabs = lora ? R->tile_nslabs : nullptr;
    a.tile_slab = lora ? R->tile_slab : nullptr;
    a.slab_cap = lora ? R->slab_cap : 0;
    a.status = L.status;
    a.overlap_prev = (after_shrink && lora) ? 1 : 0;
    a.ln_g = lin.ln_g; a.ln_stats = ln_stats;
    a.tma_store = (tm_y != nullptr && epi != EPI_PATCH) ? 1 : 0;
    const CUtensorMap& tt = lora ? *tm_t : tm_x;      // placeholders are never dereferenced
    const CUtensorMap& ty = a.tma_store ? *tm_y : tm_x;
    if (lin.has_tm_half && n_sms >= 2 && (epi != EPI_RESIDUAL || a.tma_store)) {
        a.m_tiles = (rows + 2 * BM - 1) / (2 * BM);       // 256-row tiles
        a.n_tiles = lin.n_out / P_BN;
        return launch_gemm_pair_epi(L, tm_x, lin.tm_w_half, tt, lora ? lin.tm_bt_half : lin.tm_w_half, ty, a, n_sms);
    }
    const CUtensorMap& tb = lora ? lin.tm_bt : lin.tm_w;
    if (bn == 256) return launch_gemm_epi<256>(L, tm_x, lin.tm_w, tt, tb, ty, a, n_sms);
    return launch_gemm_epi<128>(L, tm_x, lin.tm_w, tt, tb, ty, a, n_sms);
}
