// Memory-bound and small kernels of the Polymorph forward path: LayerNorm, patch gather, CLS rows,
// segmented heads + sigmoid + merge, Algorithm 2 selection, and the plain CUDA-core kernels of
// the fp32 debug build (linear with unmerged LoRA terms, attention).
#include <algorithm>
#include <atomic>

#include "common.cuh"

#define BUMP(L) do { if ((L).launches) ++*(L).launches; } while (0)

// ---------------------------------------------------------------------------------------
// element helpers
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

template <typename T> struct Vec16 { static constexpr int N = 16 / sizeof(T); };

template <typename T>
__device__ __forceinline__ void load16(const T* p, float* out) {
    uint4 raw = *reinterpret_cast<const uint4*>(p);
    if constexpr (sizeof(T) == 4) {
        out[0] = __uint_as_float(raw.x); out[1] = __uint_as_float(raw.y);
        out[2] = __uint_as_float(raw.z); out[3] = __uint_as_float(raw.w);
    } else {
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
}

template <typename T>
__device__ __forceinline__ void store16(T* p, const float* v) {
    uint4 raw;
    if constexpr (sizeof(T) == 4) {
        raw.x = __float_as_uint(v[0]); raw.y = __float_as_uint(v[1]);
        raw.z = __float_as_uint(v[2]); raw.w = __float_as_uint(v[3]);
    } else {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        raw.x = w[0]; raw.y = w[1]; raw.z = w[2]; raw.w = w[3];
    }
    *reinterpret_cast<uint4*>(p) = raw;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

// ---------------------------------------------------------------------------------------
// LayerNorm: one warp per row, 128-bit loads, the row stays in registers (d <= 1024)
// ---------------------------------------------------------------------------------------
template <typename T, typename OutT>
__device__ __forceinline__ void ln_row(const T* __restrict__ xr, const float* __restrict__ g,
                                       const float* __restrict__ b, OutT* __restrict__ yr, int d,
                                       float eps, int lane) {
    constexpr int VEC = Vec16<T>::N;
    constexpr int MAXCH = 32 / VEC;
    const int nch = d / VEC;
    float v[32];
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < MAXCH; ++i) {
        const int c = lane + 32 * i;
        if (c < nch) {
            load16<T>(xr + c * VEC, v + i * VEC);
#pragma unroll
            for (int j = 0; j < VEC; ++j) sum += v[i * VEC + j];
        } else {
#pragma unroll
            for (int j = 0; j < VEC; ++j) v[i * VEC + j] = 0.f;
        }
    }
    const float mean = warp_sum(sum) / (float)d;
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < MAXCH; ++i) {
        if (lane + 32 * i < nch) {
#pragma unroll
            for (int j = 0; j < VEC; ++j) { const float t = v[i * VEC + j] - mean; sq += t * t; }
        }
    }
    const float rstd = rsqrtf(warp_sum(sq) / (float)d + eps);
#pragma unroll
    for (int i = 0; i < MAXCH; ++i) {
        const int c = lane + 32 * i;
        if (c < nch) {
            float o[VEC];
#pragma unroll
            for (int j = 0; j < VEC; j += 4) {
                const float4 gg = *reinterpret_cast<const float4*>(g + c * VEC + j);
                const float4 bb = *reinterpret_cast<const float4*>(b + c * VEC + j);
                o[j + 0] = (v[i * VEC + j + 0] - mean) * rstd * gg.x + bb.x;
                o[j + 1] = (v[i * VEC + j + 1] - mean) * rstd * gg.y + bb.y;
                o[j + 2] = (v[i * VEC + j + 2] - mean) * rstd * gg.z + bb.z;
                o[j + 3] = (v[i * VEC + j + 3] - mean) * rstd * gg.w + bb.w;
            }
            if constexpr (sizeof(OutT) == sizeof(T)) {
                store16<OutT>(yr + c * VEC, o);
            } else {   // bf16 in, fp32 out
#pragma unroll
                for (int j = 0; j < VEC; ++j) yr[c * VEC + j] = o[j];
            }
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256) layernorm_kernel(const T* __restrict__ x,
                                                        const float* __restrict__ g,
                                                        const float* __restrict__ b,
                                                        T* __restrict__ y, int rows, int d, float eps) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    ln_row<T, T>(x + (size_t)row * d, g, b, y + (size_t)row * d, d, eps, threadIdx.x & 31);
}

// Row statistics only (mean and 1/sqrt(var + eps), biased variance, two passes over the registers):
// for the linears that have LayerNorm folded into their weights the normalised rows are never
// written out; the GEMM and shrink epilogues apply the statistics instead.
__global__ void __launch_bounds__(256) row_stats_kernel(const bf16* __restrict__ x, float2* __restrict__ stats,
                                                        int rows, int d, float eps) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    const int nch = d >> 3;
    const bf16* xr = x + (size_t)row * d;
    float v[32];
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int c = lane + 32 * i;
        if (c < nch) {
            load16<bf16>(xr + c * 8, v + i * 8);
#pragma unroll
            for (int j = 0; j < 8; ++j) sum += v[i * 8 + j];
        }
    }
    const float mean = warp_sum(sum) / (float)d;
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (lane + 32 * i < nch) {
#pragma unroll
            for (int j = 0; j < 8; ++j) { const float t = v[i * 8 + j] - mean; sq += t * t; }
        }
    }
    const float rstd = rsqrtf(warp_sum(sq) / (float)d + eps);
    if (lane == 0) stats[row] = make_float2(mean, rstd);
}

cudaError_t launch_row_stats(const Launch& L, const bf16* x, float2* stats, int rows, int d, float eps) {
    if (rows <= 0) return cudaSuccess;
    ProfScope ps(L, KC_LAYERNORM);
    row_stats_kernel<<<(rows + 7) / 8, 256, 0, L.st>>>(x, stats, rows, d, eps);
    BUMP(L);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_layernorm(const Launch& L, const T* x, const float* g, const float* b, T* y,
                             int rows, int d, float eps) {
    if (rows <= 0) return cudaSuccess;
    ProfScope ps(L, KC_LAYERNORM);
    layernorm_kernel<T><<<(rows + 7) / 8, 256, 0, L.st>>>(x, g, b, y, rows, d, eps);
    BUMP(L);
    return cudaGetLastError();
}
template cudaError_t launch_layernorm<float>(const Launch&, const float*, const float*, const float*, float*, int, int, float);
template cudaError_t launch_layernorm<bf16>(const Launch&, const bf16*, const float*, const float*, bf16*, int, int, float);

// ---------------------------------------------------------------------------------------
// patch gather (im2col) and CLS rows
// ---------------------------------------------------------------------------------------
// out[slot*g*g + (gy*g+gx)][c*P*P + py*P + px] = frames[perm[slot]][c][gy*P+py][gx*P+px]
template <typename T>
__global__ void __launch_bounds__(256) im2col_kernel(const T* __restrict__ frames,
                                                     const int* __restrict__ perm,
                                                     T* __restrict__ out, int n_frames, int img,
                                                     int patch) {
    constexpr int VEC = Vec16<T>::N;
    const int g = img / patch;
    const int pd = 3 * patch * patch;
    const int chunks_per_row = pd / VEC;
    const size_t total = (size_t)n_frames * g * g * chunks_per_row;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const int ch = (int)(i % chunks_per_row);
        const size_t r = i / chunks_per_row;
        const int p = (int)(r % (g * g));
        const int slot = (int)(r / (g * g));
        const int col = ch * VEC;
        const int c = col / (patch * patch);
        const int py = (col / patch) % patch;
        const int px = col % patch;                 // multiple of VEC (patch % VEC == 0)
        const int gy = p / g, gx = p % g;
        const T* src = frames + (((size_t)perm[slot] * 3 + c) * img + gy * patch + py) * img +
                       gx * patch + px;
        *reinterpret_cast<uint4*>(out + r * pd + col) = *reinterpret_cast<const uint4*>(src);
    }
}

template <typename T>
cudaError_t launch_im2col(const Launch& L, const T* frames, const int* perm, T* out, int n_frames,
                          int img, int patch) {
    const int g = img / patch;
    const size_t total = (size_t)n_frames * g * g * (3 * patch * patch / Vec16<T>::N);
    const int blocks = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    if (blocks == 0) return cudaSuccess;
    ProfScope ps(L, KC_OTHER);
    im2col_kernel<T><<<blocks, 256, 0, L.st>>>(frames, perm, out, n_frames, img, patch);
    BUMP(L);
    return cudaGetLastError();
}
template cudaError_t launch_im2col<float>(const Launch&, const float*, const int*, float*, int, int, int);
template cudaError_t launch_im2col<bf16>(const Launch&, const bf16*, const int*, bf16*, int, int, int);

template <typename T>
__global__ void cls_rows_kernel(const float* __restrict__ cls, const float* __restrict__ pos,
                                T* __restrict__ x, int n_frames, int tokens, int d) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_frames * d) return;
    const int f = i / d, c = i % d;
    x[(size_t)f * tokens * d + c] = from_f<T>(cls[c] + pos[c]);
}

template <typename T>
cudaError_t launch_cls_rows(const Launch& L, const float* cls, const float* pos, T* x, int n_frames,
                            int tokens, int d) {
    ProfScope ps(L, KC_OTHER);
    cls_rows_kernel<T><<<(n_frames * d + 255) / 256, 256, 0, L.st>>>(cls, pos, x, n_frames, tokens, d);
    BUMP(L);
    return cudaGetLastError();
}
template cudaError_t launch_cls_rows<float>(const Launch&, const float*, const float*, float*, int, int, int);
template cudaError_t launch_cls_rows<bf16>(const Launch&, const float*, const float*, bf16*, int, int, int);

// ---------------------------------------------------------------------------------------
// fp32 debug build: linear with unmerged LoRA terms on CUDA cores
// ---------------------------------------------------------------------------------------
// t32[row][p*RS + j] = s_a * sum_k x[row,k] A_a[k,j],  a = p-th adapter of the row's frame
template <typename T>
__global__ void __launch_bounds__(128) naive_shrink_kernel(const T* __restrict__ x, const T* __restrict__ At,
                                    const int* __restrict__ slot_off, const int* __restrict__ slot_ids,
                                    const float* __restrict__ scale, int k_in, int tokens, int RS,
                                    int max_set, float* __restrict__ t32) {
    const int row = blockIdx.x;
    const int slot = row / tokens;
    const int n = slot_off[slot + 1] - slot_off[slot];
    const T* xr = x + (size_t)row * k_in;
    for (int i = threadIdx.x; i < max_set * RS; i += blockDim.x) {
        const int p = i / RS, j = i % RS;
        float acc = 0.f;
        if (p < n) {
            const int a = slot_ids[slot_off[slot] + p];
            const T* ar = At + ((size_t)a * RS + j) * k_in;
            for (int k = 0; k < k_in; ++k) acc = fmaf(to_f(xr[k]), to_f(ar[k]), acc);
            acc *= scale[a];
        }
        t32[(size_t)row * max_set * RS + i] = acc;
    }
}

__device__ __forceinline__ float gelu_erf(float v) {
    return 0.5f * v * (1.f + erff(v * 0.70710678118654752440f));
}

template <typename T>
__global__ void __launch_bounds__(256) naive_linear_kernel(const T* __restrict__ x, const T* __restrict__ Wt,
                                    const float* __restrict__ bias, const float* __restrict__ t32,
                                    const T* __restrict__ Bt, const int* __restrict__ slot_off,
                                    const int* __restrict__ slot_ids, int rows, int k_in, int n_out,
                                    int tokens, int RS, int max_set, int slabs_max, int epi,
                                    const T* __restrict__ residual, PatchEpi pe, T* __restrict__ y) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int row = blockIdx.y;
    if (n >= n_out || row >= rows) return;
    const T* xr = x + (size_t)row * k_in;
    const T* wr = Wt + (size_t)n * k_in;
    float acc = 0.f;
    for (int k = 0; k < k_in; ++k) acc = fmaf(to_f(xr[k]), to_f(wr[k]), acc);
    acc += bias[n];
    if (t32 != nullptr) {
        const int slot = row / tokens;
        const int cnt = slot_off[slot + 1] - slot_off[slot];
        for (int p = 0; p < cnt; ++p) {
            const int a = slot_ids[slot_off[slot] + p];
            const float* tr = t32 + ((size_t)row * max_set + p) * RS;
            float d = 0.f;
            for (int j = 0; j < RS; ++j)
                d = fmaf(tr[j], to_f(Bt[(((size_t)a * slabs_max + (j >> 4)) * n_out + n) * PM_SLAB + (j & 15)]), d);
            acc += d;
        }
    }
    size_t orow = row;
    if (epi == EPI_GELU) acc = gelu_erf(acc);
    else if (epi == EPI_RESIDUAL) acc += to_f(residual[(size_t)row * n_out + n]);
    else if (epi == EPI_PATCH) {
        const int p = row % pe.g2;
        orow = (size_t)(row / pe.g2) * pe.tokens + 1 + p;
        acc += pe.pos[(size_t)(1 + p) * n_out + n];
    }
    y[orow * n_out + n] = from_f<T>(acc);
}

template <typename T>
cudaError_t launch_naive_linear(const Launch& L, const LinearDev& lin, const RouteDev& R,
                                const AdapterMeta& meta, int slabs_max, const T* x, int rows,
                                int tokens_per_frame, float* t32, int epi, const T* residual,
                                const PatchEpi& pe, T* y) {
    if (rows <= 0) return cudaSuccess;
    ProfScope ps(L, KC_GEMM);
    const int RS = slabs_max * PM_SLAB;
    const bool lora = (t32 != nullptr) && lin.lora.At != nullptr && R.max_set > 0;
    if (lora) {
        naive_shrink_kernel<T><<<rows, 128, 0, L.st>>>(x, (const T*)lin.lora.At, R.slot_off, R.slot_ids,
                                                      meta.scale, lin.k_in, tokens_per_frame, RS,
                                                      R.max_set, t32);
        BUMP(L);
    }
    dim3 grid((lin.n_out + 255) / 256, rows);
    naive_linear_kernel<T><<<grid, 256, 0, L.st>>>(x, (const T*)lin.Wt, lin.bias, lora ? t32 : nullptr,
                                                  (const T*)lin.lora.Bt, R.slot_off, R.slot_ids, rows,
                                                  lin.k_in, lin.n_out, tokens_per_frame, RS, R.max_set,
                                                  slabs_max, epi, residual, pe, y);
    BUMP(L);
    return cudaGetLastError();
}
template cudaError_t launch_naive_linear<float>(const Launch&, const LinearDev&, const RouteDev&, const AdapterMeta&, int, const float*, int, int, float*, int, const float*, const PatchEpi&, float*);
template cudaError_t launch_naive_linear<bf16>(const Launch&, const LinearDev&, const RouteDev&, const AdapterMeta&, int, const bf16*, int, int, float*, int, const bf16*, const PatchEpi&, bf16*);

// ---------------------------------------------------------------------------------------
// plain attention (any token count): one warp per query row
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) attention_simple_kernel(const T* __restrict__ qkv, T* __restrict__ out,
                                                               int tokens, int heads) {
    extern __shared__ float probs[];             // [8][tokens]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int f = blockIdx.y / heads, h = blockIdx.y % heads;
    const int qi = blockIdx.x * 8 + warp;
    if (qi >= tokens) return;
    const int d = heads * 64;
    const size_t base = (size_t)f * tokens * 3 * d;
    const T* qrow = qkv + base + (size_t)qi * 3 * d + h * 64;
    float q[64];
#pragma unroll
    for (int i = 0; i < 64; i += Vec16<T>::N) load16<T>(qrow + i, q + i);
    float* pr = probs + warp * tokens;
    float mx = -INFINITY;
    for (int j = lane; j < tokens; j += 32) {
        const T* krow = qkv + base + (size_t)j * 3 * d + d + h * 64;
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 64; i += Vec16<T>::N) {
            float kv[Vec16<T>::N];
            load16<T>(krow + i, kv);
#pragma unroll
            for (int e = 0; e < Vec16<T>::N; ++e) s = fmaf(q[i + e], kv[e], s);
        }
        s *= 0.125f;
        pr[j] = s;
        mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int j = lane; j < tokens; j += 32) {
        const float e = expf(pr[j] - mx);
        pr[j] = e;
        sum += e;
    }
    sum = warp_sum(sum);
    __syncwarp();
    float a0 = 0.f, a1 = 0.f;
    for (int j = 0; j < tokens; ++j) {
        const T* vrow = qkv + base + (size_t)j * 3 * d + 2 * d + h * 64 + 2 * lane;
        const float p = pr[j];
        a0 = fmaf(p, to_f(vrow[0]), a0);
        a1 = fmaf(p, to_f(vrow[1]), a1);
    }
    T* o = out + ((size_t)f * tokens + qi) * d + h * 64 + 2 * lane;
    o[0] = from_f<T>(a0 / sum);
    o[1] = from_f<T>(a1 / sum);
}

template <typename T>
cudaError_t launch_attention_simple(const Launch& L, const T* qkv, T* out, int n_frames, int tokens,
                                    int heads) {
    if (n_frames <= 0) return cudaSuccess;
    ProfScope ps(L, KC_ATTENTION);
    dim3 grid((tokens + 7) / 8, n_frames * heads);
    attention_simple_kernel<T><<<grid, 256, 8 * tokens * sizeof(float), L.st>>>(qkv, out, tokens, heads);
    BUMP(L);
    return cudaGetLastError();
}
template cudaError_t launch_attention_simple<float>(const Launch&, const float*, float*, int, int, int);
template cudaError_t launch_attention_simple<bf16>(const Launch&, const bf16*, bf16*, int, int, int);

// ---------------------------------------------------------------------------------------
// branched forward (Fig. 2b): the rows a frame has after the shared trunk are copied to the slots
// of its adapter branches.  Source slots lie below first_slot, destinations at or above it.
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) fanout_rows_kernel(T* __restrict__ x, const int* __restrict__ src_slot,
                                                          int first_slot, size_t slot_vec) {
    const int slot = first_slot + blockIdx.y;
    const uint4* s = reinterpret_cast<const uint4*>(x) + (size_t)src_slot[slot] * slot_vec;
    uint4* o = reinterpret_cast<uint4*>(x) + (size_t)slot * slot_vec;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < slot_vec; i += (size_t)gridDim.x * blockDim.x)
        o[i] = s[i];
}

template <typename T>
cudaError_t launch_fanout_rows(const Launch& L, T* x, const int* src_slot, int first_slot, int n_slots,
                               int tokens, int d) {
    if (n_slots <= first_slot) return cudaSuccess;
    const size_t slot_vec = (size_t)tokens * d * sizeof(T) / 16;     // d is a multiple of 64
    ProfScope ps(L, KC_OTHER);
    dim3 grid((unsigned)std::min<size_t>((slot_vec + 255) / 256, 64), n_slots - first_slot);
    fanout_rows_kernel<T><<<grid, 256, 0, L.st>>>(x, src_slot, first_slot, slot_vec);
    BUMP(L);
    return cudaGetLastError();
}
template cudaError_t launch_fanout_rows<float>(const Launch&, float*, const int*, int, int, int, int);
template cudaError_t launch_fanout_rows<bf16>(const Launch&, bf16*, const int*, int, int, int, int);

// ---------------------------------------------------------------------------------------
// final LayerNorm on the CLS rows, base head, segmented adapter heads + sigmoid + merge
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) final_ln_kernel(const T* __restrict__ x, const float* __restrict__ g,
                                                       const float* __restrict__ b, float* __restrict__ z,
                                                       int n_frames, int tokens, int d, float eps) {
    const int slot = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (slot >= n_frames) return;
    ln_row<T, float>(x + (size_t)slot * tokens * d, g, b, z + (size_t)slot * d, d, eps, threadIdx.x & 31);
}

template <typename T>
__device__ __forceinline__ float dot_row(const float* __restrict__ z, const T* __restrict__ w, int d,
                                         int lane) {
    constexpr int VEC = Vec16<T>::N;
    float acc = 0.f;
    for (int c = lane * VEC; c < d; c += 32 * VEC) {
        float wv[VEC];
        load16<T>(w + c, wv);
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc = fmaf(z[c + e], wv[e], acc);
    }
    return warp_sum(acc);
}

__device__ __forceinline__ float sigmoidf_acc(float v) { return 1.f / (1.f + expf(-v)); }

// grid (ceil(K/32), ceil(F/8)): a block owns 32 classes x 8 slots.  The 8 CLS features are staged once in
// shared memory and shared by the block's 8 warps (read straight from global memory, every class of a
// block would fetch them again: F x K x d x 4 bytes of cache traffic in all); each warp takes four of the
// classes in turn, keeps the weight row of the class in registers and walks the slots (the next class's
// row is fetched while this one is multiplied).  base_out rows are in the caller's order.
// NV = ceil(d / 32) values per lane; the dot product runs in four chains.
constexpr int BASE_HEAD_FRAMES = 8;
constexpr int BASE_HEAD_CLASSES = 32;
template <typename T, int NV>
__global__ void __launch_bounds__(256) base_head_kernel(const float* __restrict__ z, const T* __restrict__ wt,
                                                        const float* __restrict__ bias,
                                                        const int* __restrict__ perm, int d, int n_classes,
                                                        int n_frames, float* __restrict__ base_out) {
    __shared__ float zs[BASE_HEAD_FRAMES][NV * 32];
    const int s0 = blockIdx.y * BASE_HEAD_FRAMES, ns = min(n_frames - s0, BASE_HEAD_FRAMES);
    for (int i = threadIdx.x; i < BASE_HEAD_FRAMES * NV * 32; i += 256) {
        const int sl = i / (NV * 32), c = i % (NV * 32);
        zs[sl][c] = (sl < ns && c < d) ? z[(size_t)(s0 + sl) * d + c] : 0.f;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    auto fetch = [&](int k, float (&w)[NV]) {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const int c = lane + 32 * i;
            w[i] = (k < n_classes && c < d) ? to_f(wt[(size_t)k * d + c]) : 0.f;
        }
    };
    const int k0 = blockIdx.x * BASE_HEAD_CLASSES + (threadIdx.x >> 5);
    float w[NV], wn[NV];
    fetch(k0, w);
    for (int k = k0; k < n_classes && k < (int)(blockIdx.x + 1) * BASE_HEAD_CLASSES; k += 8) {
        fetch(k + 8 < (int)(blockIdx.x + 1) * BASE_HEAD_CLASSES ? k + 8 : n_classes, wn);
        const float bk = bias[k];
        for (int sl = 0; sl < ns; ++sl) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < NV; ++i) acc[i & 3] = fmaf(zs[sl][lane + 32 * i], w[i], acc[i & 3]);
            const float dot = warp_sum((acc[0] + acc[1]) + (acc[2] + acc[3]));
            if (lane == 0) base_out[(size_t)perm[s0 + sl] * n_classes + k] = sigmoidf_acc(dot + bk);
        }
#pragma unroll
        for (int i = 0; i < NV; ++i) w[i] = wn[i];
    }
}

// grid (max_set, F): block = the p-th active adapter of one slot; its warps walk the adapter's
// class list.  Scores are positive, so the maximum over adapters is an integer atomicMax on the
// float bit pattern of a zero-initialised row (order-free, hence deterministic).
template <typename T>
__global__ void __launch_bounds__(256) adapter_heads_kernel(const float* __restrict__ z, const T* __restrict__ hcat,
                                                            const float* __restrict__ hbias,
                                                            const int* __restrict__ hcls,
                                                            const int* __restrict__ hoff,
                                                            const int* __restrict__ slot_off,
                                                            const int* __restrict__ slot_ids,
                                                            const int* __restrict__ perm, int d,
                                                            int n_classes, float* __restrict__ scores) {
    const int slot = blockIdx.y, p = blockIdx.x;
    if (p >= slot_off[slot + 1] - slot_off[slot]) return;
    const int a = slot_ids[slot_off[slot] + p];
    const int lane = threadIdx.x & 31;
    for (int r = hoff[a] + (threadIdx.x >> 5); r < hoff[a + 1]; r += 8) {
        const float v = dot_row<T>(z + (size_t)slot * d, hcat + (size_t)r * d, d, lane) + hbias[r];
        if (lane == 0)
            atomicMax(reinterpret_cast<int*>(scores + (size_t)perm[slot] * n_classes + hcls[r]),
                      __float_as_int(sigmoidf_acc(v)));
    }
}

template <typename T>
cudaError_t launch_heads(const Launch& L, const T* x, int n_slots, int n_out_frames, int n_base_slots,
                         int tokens, int d, float eps,
                         const float* lnf_g, const float* lnf_b, float* z,
                         const T* base_wt, const float* base_b, int n_classes,
                         const T* hcat, const float* hbias, const int* hcls, const int* hoff,
                         const RouteDev& R, float* scores_out, float* base_out) {
    if (n_slots <= 0) return cudaSuccess;
    ProfScope ps(L, KC_HEADS);
    final_ln_kernel<T><<<(n_slots + 7) / 8, 256, 0, L.st>>>(x, lnf_g, lnf_b, z, n_slots, tokens, d, eps);
    BUMP(L);
    if (base_out && n_base_slots > 0) {
        dim3 grid((n_classes + BASE_HEAD_CLASSES - 1) / BASE_HEAD_CLASSES, (n_base_slots + BASE_HEAD_FRAMES - 1) / BASE_HEAD_FRAMES);
        const int nv = (d + 31) / 32;                  // d <= 1024
        auto kern = nv <= 6 ? base_head_kernel<T, 6> : nv <= 12 ? base_head_kernel<T, 12>
                  : nv <= 24 ? base_head_kernel<T, 24> : base_head_kernel<T, 32>;
        kern<<<grid, 256, 0, L.st>>>(z, base_wt, base_b, R.perm, d, n_classes, n_base_slots, base_out);
        BUMP(L);
    }
    cudaError_t e = cudaMemsetAsync(scores_out, 0, (size_t)n_out_frames * n_classes * sizeof(float), L.st);
    if (e != cudaSuccess) return e;
    if (R.max_set > 0) {
        dim3 grid(R.max_set, n_slots);
        adapter_heads_kernel<T><<<grid, 256, 0, L.st>>>(z, hcat, hbias, hcls, hoff, R.slot_off, R.slot_ids,
                                                       R.perm, d, n_classes, scores_out);
        BUMP(L);
    }
    return cudaGetLastError();
}
template cudaError_t launch_heads<float>(const Launch&, const float*, int, int, int, int, int, float, const float*, const float*, float*, const float*, const float*, int, const float*, const float*, const int*, const int*, const RouteDev&, float*, float*);
template cudaError_t launch_heads<bf16>(const Launch&, const bf16*, int, int, int, int, int, float, const float*, const float*, float*, const bf16*, const float*, int, const bf16*, const float*, const int*, const int*, const RouteDev&, float*, float*);

// ---------------------------------------------------------------------------------------
// Algorithm 2 on the device: one warp per frame, any number of blocks
// ---------------------------------------------------------------------------------------
// The greedy branch visits contexts by (size, id) and takes a context iff it provides a still
// uncovered label; that set equals { first(l) : l in Y_t }, first(l) being the first provider of l
// in visiting order, so it reduces to a table lookup and a bit-mask OR.
// Phase 1 (all blocks): threshold -> label bit set -> keep / copy / greedy -> adapter bit mask and
// its population count per frame.  Phase 2 (the block that finishes last, found with a counter in
// the scratch area): prefix sum of the counts and emission of the sorted id lists.  `scratch` holds
// the counter in word 0 (zero between launches; its place does not depend on the frame count, so
// calls with different batch sizes may follow each other on one scratch area) and, from word 1 on,
// n_frames * ceil(n_adapters/64) mask words.  Adapter ids read from prev_ids / first that fall
// outside [0, n_adapters) are skipped and reported as PM_ERR_ARG in the status word.
constexpr int SELECT_THREADS = 256;

__global__ void __launch_bounds__(SELECT_THREADS) select_kernel(const float* __restrict__ scores, int n_frames,
                                                      int n_classes, int n_adapters, float thr,
                                                      int context_copy, int has_prev,
                                                      uint32_t* __restrict__ prev_labels,
                                                      const int* __restrict__ prev_off,
                                                      const int* __restrict__ prev_ids,
                                                      const int* __restrict__ first,
                                                      const uint64_t* __restrict__ provider,
                                                      uint64_t* scratch,
                                                      int* next_off,
                                                      int* __restrict__ next_ids, int ids_capacity,
                                                      int* __restrict__ status,
                                                      unsigned long long* __restrict__ metrics) {
    __shared__ int partial[SELECT_THREADS];
    __shared__ int is_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = SELECT_THREADS >> 5;
    const int NW = (n_classes + 31) / 32;
    const int AW = (n_adapters + 63) / 64;     // <= 4 (checked on the host)
    unsigned int* done = reinterpret_cast<unsigned int*>(scratch);
    uint64_t* masks = scratch + 1;

    const int f = blockIdx.x * nwarps + warp;
    if (f < n_frames) {
        uint64_t prev_mask[4] = {0, 0, 0, 0}, greedy[4] = {0, 0, 0, 0};
        if (has_prev) {
            // a valid S_{t-1} has at most n_adapters distinct ids; anything else is a caller error
            const int p0 = prev_off[f];
            int pn = prev_off[f + 1] - p0;
            if (p0 < 0 || pn < 0 || pn > n_adapters) {
                if (lane == 0) atomicCAS(status, 0, (int)PM_ERR_ARG);
                pn = 0;
            }
            for (int i = lane; i < pn; i += 32) {
                const int a = prev_ids[p0 + i];
                if ((unsigned)a < (unsigned)n_adapters) prev_mask[a >> 6] |= 1ull << (a & 63);
                else atomicCAS(status, 0, (int)PM_ERR_ARG);
            }
#pragma unroll
            for (int w = 0; w < 4; ++w) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) prev_mask[w] |= __shfl_xor_sync(0xFFFFFFFFu, prev_mask[w], o);
            }
        }
        bool same = true, covered = true;
        for (int w0 = 0; w0 < NW; w0 += 8) {
            float sc[8];
            uint32_t old[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {               // eight independent loads in flight
                const int k = (w0 + i) * 32 + lane;
                sc[i] = (w0 + i < NW && k < n_classes) ? scores[(size_t)f * n_classes + k] : -INFINITY;
                old[i] = (has_prev && prev_labels && w0 + i < NW && lane == 0) ? prev_labels[(size_t)f * NW + w0 + i] : 0u;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int w = w0 + i;
                if (w >= NW) break;
                const int k = w * 32 + lane;
                const bool on = sc[i] > thr;
                const uint32_t word = __ballot_sync(0xFFFFFFFFu, on);
                if (prev_labels && lane == 0) {
                    if (has_prev && old[i] != word) same = false;
                    prev_labels[(size_t)f * NW + w] = word;
                }
                if (on) {
                    bool cov = false;
                    for (int q = 0; q < AW; ++q) cov |= (provider[(size_t)k * AW + q] & prev_mask[q]) != 0;
                    if (!cov) covered = false;
                    const int a = first[k];                 // -1: nobody provides this label
                    if ((unsigned)a < (unsigned)n_adapters) greedy[a >> 6] |= 1ull << (a & 63);
                    else if (a != -1) atomicCAS(status, 0, (int)PM_ERR_ARG);
                }
            }
        }
        covered = __all_sync(0xFFFFFFFFu, covered);
        same = __all_sync(0xFFFFFFFFu, same);
#pragma unroll
        for (int w = 0; w < 4; ++w) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) greedy[w] |= __shfl_xor_sync(0xFFFFFFFFu, greedy[w], o);
        }
        const bool keep = has_prev && ((prev_labels != nullptr && same) || (context_copy && covered));
        int cnt = 0;
        bool changed = false;
        for (int q = 0; q < AW; ++q) {
            const uint64_t m = keep ? prev_mask[q] : greedy[q];
            cnt += __popcll(m);
            changed |= m != prev_mask[q];
            if (lane == 0) masks[(size_t)f * AW + q] = m;
        }
        if (lane == 0) next_off[f + 1] = cnt;
        // Eq. 8: one switch per stream and step whose chosen set differs from the previous one
        if (lane == 0 && metrics && has_prev && changed) atomicAdd(metrics + 2, 1ull);
    }
    // ---- the last block to arrive here does the scan and the emission
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(done, 1u) == gridDim.x - 1) ? 1 : 0;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    volatile int* voff = next_off;
    volatile uint64_t* vmasks = masks;
    // exclusive scan of the counts: each thread owns a contiguous chunk of frames
    const int per = (n_frames + SELECT_THREADS - 1) / SELECT_THREADS;
    const int lo = min(n_frames, (int)threadIdx.x * per), hi = min(n_frames, lo + per);
    int s = 0;
    for (int g = lo; g < hi; ++g) s += voff[g + 1];
    partial[threadIdx.x] = s;
    __syncthreads();
    for (int o = 1; o < SELECT_THREADS; o <<= 1) {
        const int v = (int)threadIdx.x >= o ? partial[threadIdx.x - o] : 0;
        __syncthreads();
        partial[threadIdx.x] += v;
        __syncthreads();
    }
    int run = partial[threadIdx.x] - s;        // exclusive prefix of this chunk
    if (threadIdx.x == 0) { voff[0] = 0; *done = 0u; }
    if (threadIdx.x == SELECT_THREADS - 1 && metrics) {
        // Eq. 7: frames seen and active contexts chosen (their ratio is AvgCoverage)
        atomicAdd(metrics + 0, (unsigned long long)n_frames);
        atomicAdd(metrics + 1, (unsigned long long)partial[threadIdx.x]);
    }
    for (int g = lo; g < hi; ++g) {
        run += voff[g + 1];
        voff[g + 1] = run;
    }
    __syncthreads();
    // emission: one thread per frame (all frames' loads are in flight at once; a frame has few ids)
    for (int g = threadIdx.x; g < n_frames; g += SELECT_THREADS) {
        int pos = voff[g];
        for (int q = 0; q < AW; ++q) {
            uint64_t m = vmasks[(size_t)g * AW + q];
            while (m) {
                const int b = __ffsll((long long)m) - 1;
                m &= m - 1;
                if (pos < ids_capacity) next_ids[pos] = q * 64 + b;
                else atomicCAS(status, 0, (int)PM_ERR_CAPACITY);
                ++pos;
            }
        }
    }
}

cudaError_t launch_select(const Launch& L, const float* scores, int n_frames, int n_classes,
                          int n_adapters, float thr, int context_copy, int has_prev,
                          uint32_t* prev_labels, const int* prev_off, const int* prev_ids,
                          const int* first, const uint64_t* provider, uint64_t* mask_scratch,
                          int* next_off, int* next_ids, int ids_capacity, unsigned long long* metrics) {
    ProfScope ps(L, KC_SELECT);
    const int blocks = n_frames > 0 ? (n_frames + SELECT_THREADS / 32 - 1) / (SELECT_THREADS / 32) : 1;
    select_kernel<<<blocks, SELECT_THREADS, 0, L.st>>>(scores, n_frames, n_classes, n_adapters, thr, context_copy,
                                        has_prev, prev_labels, prev_off, prev_ids, first, provider,
                                        mask_scratch, next_off, next_ids, ids_capacity, L.status, metrics);
    BUMP(L);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// pm_select_static: Algorithm 2 selection for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------
// select_kernel needs one scratch word list per frame (the chosen adapter bit masks, written in its
// first phase and read back after the prefix sum).  pm_select takes that scratch from the handle,
// which allocates it; this variant keeps it in the library image instead, so a caller that is
// forbidden to call cudaMalloc (a real-time loop with a no-allocation rule, a plugin running
// inside another framework's memory pool, a process whose device memory is fully pre-assigned)
// can still run the selection.  Every GPU that loads the library carries the array until exit.
#define PM_SELECT_STATIC_WORDS (PM_SELECT_STATIC_MAX_FRAMES * (PM_SELECT_STATIC_MAX_ADAPTERS / 64))

static __device__ __align__(256) unsigned long long pm_select_static_masks[1 + PM_SELECT_STATIC_WORDS];   // block counter, then the masks
static __device__ __align__(256) int pm_select_static_status[64];   // word 0: status when the caller passes none

namespace {
constexpr int STATIC_MAX_DEVICES = 64;
struct StaticScratch { uint64_t* masks; int* status; };
StaticScratch g_static_scratch[STATIC_MAX_DEVICES];       // device addresses, per device ordinal
// set (release) once a device's addresses are stored; host threads that see it (acquire) may use them.
// Two threads racing through the first call on a device both look the addresses up and store the
// same values.
std::atomic<bool> g_static_ready[STATIC_MAX_DEVICES];
}  // namespace

extern "C" int pm_select_static(const float* scores, int n_frames, int n_classes, int n_adapters,
                                float score_thr, int context_copy, int has_prev, uint32_t* prev_labels,
                                const int32_t* prev_offsets, const int32_t* prev_ids,
                                const int32_t* first, const uint64_t* provider,
                                int32_t* next_offsets, int32_t* next_ids, int ids_capacity,
                                int32_t* status_out, void* cuda_stream) {
    if (n_frames < 0 || n_classes <= 0 || n_adapters <= 0 || !scores || !first || !provider ||
        !next_offsets || ids_capacity < 0 || (!next_ids && ids_capacity > 0))
        return PM_ERR_ARG;
    if (has_prev && (!prev_labels || !prev_offsets || !prev_ids)) return PM_ERR_ARG;
    if (n_frames > PM_SELECT_STATIC_MAX_FRAMES || n_adapters > PM_SELECT_STATIC_MAX_ADAPTERS)
        return PM_ERR_CAPACITY;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) return PM_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (st != nullptr && st != cudaStreamLegacy && st != cudaStreamPerThread) {
        // the scratch array is per device: the stream must belong to the current one
        int sdev = -1;
        if (cudaStreamGetDevice(st, &sdev) != cudaSuccess) { cudaGetLastError(); return PM_ERR_CUDA; }
        if (sdev != dev) return PM_ERR_ARG;
    }
    if (!g_static_ready[dev].load(std::memory_order_acquire)) {
        // The array's name is only a host-side stand-in here: ask the runtime for the device address
        // of this device's copy (the current device is the one the stream belongs to).
        void *m = nullptr, *s = nullptr;
        if (cudaGetSymbolAddress(&m, pm_select_static_masks) != cudaSuccess ||
            cudaGetSymbolAddress(&s, pm_select_static_status) != cudaSuccess || !m || !s) {
            cudaGetLastError();
            return PM_ERR_CUDA;
        }
        g_static_scratch[dev].masks = static_cast<uint64_t*>(m);
        g_static_scratch[dev].status = static_cast<int*>(s);
        g_static_ready[dev].store(true, std::memory_order_release);
    }
    int* status = status_out ? status_out : g_static_scratch[dev].status;
    // what must start at zero: the status word and the kernel's block counter (word 0 of the array);
    // the mask words themselves are all rewritten before they are read
    if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess ||
        cudaMemsetAsync(g_static_scratch[dev].masks, 0, sizeof(uint64_t), st) != cudaSuccess)
        return PM_ERR_CUDA;
    Launch L;
    L.st = st;
    L.status = status;
    if (launch_select(L, scores, n_frames, n_classes, n_adapters, score_thr, context_copy, has_prev,
                      prev_labels, prev_offsets, prev_ids, first, provider, g_static_scratch[dev].masks,
                      next_offsets, next_ids, ids_capacity) != cudaSuccess)
        return PM_ERR_CUDA;
    return PM_OK;
}
