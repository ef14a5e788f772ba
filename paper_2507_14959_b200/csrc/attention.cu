// Attention of the bf16 build: softmax(q k^T / 8) v per (frame, head), head dim 64.
//
// One CTA owns one (frame, head) (or a slice of its query rows when there are more than 256):
// K and V of the head are staged once in shared memory (16-byte chunks XOR-swizzled by row so
// that ldmatrix is conflict-free), each warp owns 16 query rows and walks the keys in blocks of
// 64 with an online softmax in fp32; both contractions run on the tensor cores
// (mma.sync m16n8k16, bf16 in, fp32 accumulate).  Key blocks are trimmed to the 8-key tile, so
// 197 tokens cost 200 key columns, not 256.
#include "common.cuh"

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

}  // namespace

cudaError_t launch_attention_mma(const Launch& L, const bf16* qkv, bf16* out, int n_frames, int tokens,
                                 int heads) {
    if (n_frames <= 0) return cudaSuccess;
    const int groups = (tokens + 15) / 16;
    const int slices = (groups + 15) / 16;
    const int warps = (groups + slices - 1) / slices;
    const int tpad = groups * 16;
    const size_t smem = (size_t)tpad * 256;
    if (smem > 227 * 1024) return launch_attention_simple<bf16>(L, qkv, out, n_frames, tokens, heads);
    static size_t smem_set = 0;
    if (smem > smem_set) {
        cudaError_t e = cudaFuncSetAttribute(attention_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        smem_set = smem;
    }
    ProfScope ps(L, KC_ATTENTION);
    dim3 grid(slices, n_frames * heads);
    attention_mma_kernel<<<grid, warps * 32, smem, L.st>>>(qkv, out, tokens, heads, tpad, warps * 16);
    BUMP(L);
    return cudaGetLastError();
}
