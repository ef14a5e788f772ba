// Shared declarations of the Polymorph B200 library (host structures, launch prototypes).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <string>
#include <vector>

#include "polymorph.h"

typedef __nv_bfloat16 bf16;

#define PM_TILE_M 128          // rows of one GEMM tile
#define PM_SLAB 16             // LoRA ranks are handled in slabs of 16 (one UMMA K step)

// ---------------------------------------------------------------------------------------
// device-side views
// ---------------------------------------------------------------------------------------
// LoRA arenas of one linear.  At: [max_adapters * RS, k_in] (row a*RS + j = column j of A_a),
// Bt: [max_adapters * slabs_max][n_out][16] (Bt[a*slabs_max + s][n][j] = B_a[16 s + j, n]);
// RS = slabs_max * 16.  Unused ranks and unregistered adapters are zero.
struct LoraArena {
    void* At = nullptr;
    void* Bt = nullptr;
};

struct LinearDev {
    int k_in = 0, n_out = 0;
    void* Wt = nullptr;        // [n_out, k_in]  (W transposed: K-major for the tensor cores)
    float* bias = nullptr;     // [n_out]
    LoraArena lora;
    // tensor maps of the static operands (bf16 build only)
    CUtensorMap tm_w, tm_at, tm_bt;
    bool has_tm = false;
    // n_out a multiple of 256: boxes of 128 output columns for the CTA-pair GEMM
    CUtensorMap tm_w_half, tm_bt_half;
    bool has_tm_half = false;
    // LayerNorm folded into this linear (its input is the raw residual stream x, not LN(x)):
    //   LN(x) W + b = rstd (x W' - mu g) + b',  W' = gamma o W,  g[n] = sum_k W'[k,n],  b' = b + beta W
    // Wt / bias above then hold W' / b'; the LoRA arena holds A' = gamma o A and, per arena rank j,
    //   ln_c1[j] = sum_k A'[k,j],  ln_c2[j] = sum_k beta[k] A[k,j].
    const float* ln_g = nullptr;       // [n_out], null = not folded
    const float* ln_c1 = nullptr;      // [max_adapters * RS]
    const float* ln_c2 = nullptr;
};

// Per-batch routing of frames to adapters, in SLOT order (slot = position after bucketing
// frames by adapter set).  All arrays live on the device.
struct RouteDev {
    int n_frames = 0, tokens = 0, n_tiles = 0, slab_cap = 0, max_set = 0;
    int* perm = nullptr;        // [F] slot -> caller's frame index
    int* slot_off = nullptr;    // [F+1] CSR over slots
    int* slot_ids = nullptr;    // [nnz] ascending adapter ids per slot
    int* src_slot = nullptr;    // [F] branched forward only: the trunk slot whose rows a branch slot copies
    // tile plan (rows 128*t .. 128*t+127).  Tiles 2p and 2p+1 carry the SAME slab list, the union of
    // what the 256 rows of the pair need (the CTA-pair GEMM applies one slab to both halves); a
    // tile's mask is zero for a slab none of its rows uses.  n_tiles is even.
    int* tile_nslabs = nullptr;     // [n_tiles]
    int* tile_slab = nullptr;       // [n_tiles, slab_cap] arena slab index a*slabs_max + s
    float* tile_scale = nullptr;    // [n_tiles, slab_cap] s_a
    uint32_t* tile_mask = nullptr;  // [n_tiles, slab_cap, 4] 128-bit mask of rows using the slab
};

struct AdapterMeta {            // device arrays indexed by adapter id
    float* scale = nullptr;     // [max_adapters]
    int* rank = nullptr;        // [max_adapters], 0 = not registered
};

enum { EPI_NONE = 0, EPI_GELU = 1, EPI_RESIDUAL = 2, EPI_PATCH = 3 };

struct PatchEpi {               // EPI_PATCH: GEMM row i = patch (i % g2) of slot (i / g2)
    int g2 = 0, tokens = 0;     //   -> output row slot*tokens + 1 + patch, plus pos[1+patch]
    const float* pos = nullptr; // [tokens, n_out] fp32
};

// ---------------------------------------------------------------------------------------
// launch prototypes (definitions in kernels_simple.cu / gemm_tcgen05.cu / attention.cu)
// every function enqueues on `st`, bumps *launches per kernel and returns a cudaError_t
// ---------------------------------------------------------------------------------------
// Optional per-kernel-class device timing (CUDA events on the launching stream).
enum { KC_GEMM = 0, KC_SHRINK = 1, KC_ATTENTION = 2, KC_LAYERNORM = 3, KC_OTHER = 4, KC_HEADS = 5, KC_SELECT = 6,
       KC_PLAN = 7, KC_COUNT = PM_PROFILE_CLASSES };
struct Profiler {
    bool on = false;
    std::vector<cudaEvent_t> ev;     // pairs: 2*i start, 2*i+1 stop
    std::vector<int> cls;            // class of pair i
    size_t used = 0;                 // pairs in use
    ~Profiler() { for (cudaEvent_t e : ev) cudaEventDestroy(e); }
};

struct Launch {
    cudaStream_t st = 0;
    long long* launches = nullptr;
    int* status = nullptr;      // device status word
    Profiler* prof = nullptr;
};

struct ProfScope {              // brackets the launches made while it is alive
    Profiler* p = nullptr;
    cudaStream_t st = 0;
    size_t idx = 0;
    ProfScope(const Launch& L, int kclass) {
        if (!L.prof || !L.prof->on) return;
        p = L.prof; st = L.st;
        if (p->used * 2 >= p->ev.size()) {
            cudaEvent_t a, b;
            if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { p = nullptr; return; }
            p->ev.push_back(a); p->ev.push_back(b); p->cls.push_back(kclass);
        }
        idx = p->used++;
        p->cls[idx] = kclass;
        cudaEventRecord(p->ev[2 * idx], st);
    }
    ~ProfScope() { if (p) cudaEventRecord(p->ev[2 * idx + 1], st); }
};

template <typename T>
cudaError_t launch_layernorm(const Launch& L, const T* x, const float* g, const float* b, T* y,
                             int rows, int d, float eps);
template <typename T>
cudaError_t launch_attention_simple(const Launch& L, const T* qkv, T* out, int n_frames, int tokens,
                                    int heads);
cudaError_t launch_attention_mma(const Launch& L, const bf16* qkv, bf16* out, int n_frames,
                                 int tokens, int heads);
// tcgen05 attention (bf16, up to 624 tokens): tensor maps over qkv [n_frames*tokens, 3*heads*64]
bool attention_tc_supported(int tokens);
bool attention_encode_maps(const bf16* qkv, int n_frames, int tokens, int heads, CUtensorMap* tm_q,
                           CUtensorMap* tm_kv);
// n_sms > 0 selects the pipelined persistent kernel where it applies (one key block); 0 = never
cudaError_t launch_attention_tc(const Launch& L, const CUtensorMap& tm_q, const CUtensorMap& tm_kv,
                                bf16* out, int n_frames, int tokens, int heads, int n_sms);
template <typename T>
cudaError_t launch_im2col(const Launch& L, const T* frames, const int* perm, T* out, int n_frames,
                          int img, int patch);
template <typename T>
cudaError_t launch_cls_rows(const Launch& L, const float* cls, const float* pos, T* x, int n_frames,
                            int tokens, int d);
// fp32 debug / reference-quality linear: t32 = scaled shrink per (row, set position, rank)
template <typename T>
cudaError_t launch_naive_linear(const Launch& L, const LinearDev& lin, const RouteDev& R,
                                const AdapterMeta& meta, int slabs_max, const T* x, int rows,
                                int tokens_per_frame, float* t32, int epi, const T* residual,
                                const PatchEpi& pe, T* y);
// tensor-core path (bf16): shrink into the slab buffer, then the fused GEMM
// A linear with LayerNorm folded in (lin.ln_g != null) needs per-row (mean, 1/sqrt(var + eps)) of x:
// either ln_stats (already computed) or stats_out (the shrink computes them from the x tiles it
// streams anyway, uses them and leaves them there for the GEMM), never both.
cudaError_t launch_shrink(const Launch& L, const LinearDev& lin, const RouteDev& R,
                          const CUtensorMap* tm_x, const bf16* x, int rows, bf16* tbuf, int n_sms,
                          const float2* ln_stats, float2* stats_out, float ln_eps);
cudaError_t launch_row_stats(const Launch& L, const bf16* x, float2* stats, int rows, int d, float eps);
// after_shrink: the kernel enqueued just before on the stream is this linear's launch_shrink; the GEMM
// may then start before it has finished (programmatic dependent launch) and awaits its results itself.
// tm_y: [rows, n_out] output map with a (32 x 32) box and 64B swizzle for the TMA-store epilogue, or
// null to store straight from registers (always the case for EPI_PATCH, whose rows are remapped)
cudaError_t launch_lora_gemm(const Launch& L, const LinearDev& lin, const RouteDev* R,
                             const CUtensorMap& tm_x, const CUtensorMap* tm_t, const CUtensorMap* tm_y,
                             int rows, int epi, const bf16* residual, const PatchEpi& pe, bf16* y,
                             int n_sms, const float2* ln_stats, bool after_shrink = false);
// x rows of slots [first_slot, n_slots) <- x rows of slot src_slot[slot] (a slot below first_slot)
template <typename T>
cudaError_t launch_fanout_rows(const Launch& L, T* x, const int* src_slot, int first_slot, int n_slots,
                               int tokens, int d);
// n_slots CLS rows are normalised and feed the adapter heads of their slot; the first n_base_slots
// also feed the base head; scores_out has n_out_frames rows (several slots may merge into one row)
template <typename T>
cudaError_t launch_heads(const Launch& L, const T* x, int n_slots, int n_out_frames, int n_base_slots,
                         int tokens, int d, float eps,
                         const float* lnf_g, const float* lnf_b, float* z,
                         const T* base_wt, const float* base_b, int n_classes,
                         const T* hcat, const float* hbias, const int* hcls, const int* hoff,
                         const RouteDev& R, float* scores_out, float* base_out);
// Builds the routing tables of R (perm, slot CSR, tile plan) on the device from a device CSR
// (plan_device.cu).  Problems found in the lists go to the status word.
cudaError_t launch_device_plan(const Launch& L, const RouteDev& R, int n_frames, int max_set, int max_adapters,
                               int slabs_max, const int* off, const int* ids, const AdapterMeta& meta);
cudaError_t launch_select(const Launch& L, const float* scores, int n_frames, int n_classes,
                          int n_adapters, float thr, int context_copy, int has_prev,
                          uint32_t* prev_labels, const int* prev_off, const int* prev_ids,
                          const int* first, const uint64_t* provider, uint64_t* mask_scratch,
                          int* next_off, int* next_ids, int ids_capacity,
                          unsigned long long* metrics = nullptr);   // [frames, sum |S_t|, switches] or null

// cudaFuncSetAttribute acts on the current device only, so "already set" is remembered per device
// ordinal: the largest dynamic shared-memory size granted to one kernel on each device.
struct SmemGrant {
    std::atomic<int> granted[64];
    template <typename Kernel>
    cudaError_t ensure(Kernel kernel, int bytes) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        std::atomic<int>& g = granted[dev & 63];
        if (bytes <= g.load(std::memory_order_acquire)) return cudaSuccess;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e != cudaSuccess) return e;
        int cur = g.load(std::memory_order_relaxed);
        while (cur < bytes && !g.compare_exchange_weak(cur, bytes, std::memory_order_release)) {}
        return cudaSuccess;
    }
};

// ---- whole-network kernel for a handful of frames (latency_kernel.cu)
// One linear as this kernel sees it (device pointers into the handle's weights and LoRA arenas).
struct LatLinear {
    CUtensorMap tm_w;          // W^T [n_out, k_in], boxes of [64 rows][64 columns], 128B swizzle
    CUtensorMap tm_at;         // A^T arena [max_adapters * RS, k_in], boxes of [16 rows][64 columns], 128B swizzle
    CUtensorMap tm_bt;         // B^T arena [max_adapters * slabs_max * n_out, 16], boxes of [128 rows][16 columns], 32B swizzle
    const bf16* Wt;            // [n_out, k_in]
    const float* bias;         // [n_out]
    const float* ln_g;         // [n_out] or null (LayerNorm folded into W)
    const bf16* At;            // [max_adapters * RS, k_in] or null
    const bf16* Bt;            // [max_adapters * slabs_max][n_out][16]
    const float* c1;           // [max_adapters * RS] (folded linears)
    const float* c2;
    uint32_t adapted[8];       // bit a: adapter a really touches this linear
    int k_in, n_out;
};

struct LatArgs {
    const bf16* frames;        // [F, 3, img, img]
    int n_frames, img, grid, tokens, tiles_pf, d, heads, mlp, layers, n_classes, patch_dim;
    int ring_slots;            // 32 KB slots of the weight ring (set by the launcher)
    float eps;
    const LatLinear* lin;      // [layers * 4 + 1]: the blocks' linears, then the patch projection
    CUtensorMap tm_kv;         // the exchange buffer as [2 * F * tokens, 2 d], boxes of [tpad rows][64 columns]
    const float *cls, *pos, *lnf_g, *lnf_b;
    const bf16* head_wt;       // [n_classes, d]
    const float* head_b;
    const bf16* hcat;          // adapter head rows [sum n_cls, d]
    const float* hbias;
    const int *hcls, *hoff;
    const int *set_off, *set_ids;          // device CSR over slots (slot s = CTA group s)
    const int* perm;                       // [F] slot -> caller's frame index, or null (slot = frame)
    int max_set, max_adapters, slabs_max;
    const int* rank;
    const float* scale;
    bf16* kv;                  // [2][F * tokens][2 d]: keys and values of the blocks, two buffers used in turn
    unsigned int* bar;         // [F] arrival counters of the frames' CTAs (cleared before every launch)
    float *scores_out, *base_out;          // [F, n_classes]
    int* status;
};

// bytes of dynamic shared memory the kernel takes for this geometry (more than any device has if it cannot run)
size_t latency_smem_bytes(int d, int mlp, int patch_dim, int tokens, int layers);
// One launch for the whole forward of a.n_frames frames; a.status is taken from L.  The grid
// (n_frames * tiles_pf CTAs, one per SM) must be resident at once: a cooperative launch, which fails
// with an error instead of starting if it cannot be.
cudaError_t launch_latency_forward(const Launch& L, const LatArgs& a);

// tensor-map helpers (gemm_tcgen05.cu); return false if the driver entry point is unavailable
bool tm_encode_2d(CUtensorMap* tm, const void* base, uint64_t inner, uint64_t outer,
                  uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, int swizzle);
bool tm_encode_3d(CUtensorMap* tm, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                  uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1,
                  uint32_t b2, int swizzle);
