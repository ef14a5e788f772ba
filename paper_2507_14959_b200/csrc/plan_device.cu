// Routing plan built on the device.
//
// The host planner (Router::build in api.cu) turns a CSR of per-frame adapter sets into the tables
// the kernels read: frames bucketed by set (perm, slot CSR) and, per 256-row pair of GEMM tiles,
// the LoRA slabs the pair needs with their scales and row masks.  When the sets were themselves
// produced on the GPU (pm_select, Algorithm 2) a host planner costs a device-to-host copy and a
// stream synchronisation per step.  The two kernels here build the same tables from a CSR that
// stays on the device, so forward -> select -> next forward runs without the host in between.
//
// The bucketing order may differ from the host planner's (any order is correct: a row's result
// does not depend on its neighbours, rows that lack an adapter get exact zeros from the masks).
#include <algorithm>
#include <climits>

#include "common.cuh"

#define BUMP(L) do { if ((L).launches) ++*(L).launches; } while (0)

namespace {

constexpr int PLAN_THREADS = 1024;

// Visits the valid, distinct ids of one frame in ascending order.  Invalid ids (out of range, not
// registered) are skipped and reported; duplicates collapse and are reported.
struct SetWalker {
    const int* ids;
    int n, max_adapters;
    const int* rank;
    int last = -1;
    __device__ SetWalker(const int* ids_, int n_, int max_adapters_, const int* rank_)
        : ids(ids_), n(n_), max_adapters(max_adapters_), rank(rank_) {}
    __device__ bool valid(int a) const { return a >= 0 && a < max_adapters && rank[a] > 0; }
    __device__ int next() {                       // -1 when exhausted
        int best = INT_MAX;
        for (int i = 0; i < n; ++i) {
            const int a = ids[i];
            if (valid(a) && a > last && a < best) best = a;
        }
        if (best == INT_MAX) return -1;
        last = best;
        return best;
    }
};

// One block.  Orders the frames by adapter set and writes perm, the slot CSR and src_slot.
__global__ void __launch_bounds__(PLAN_THREADS) plan_slots_kernel(int n_frames, int max_set, int max_adapters,
                                                                 const int* __restrict__ off,
                                                                 const int* __restrict__ ids,
                                                                 const int* __restrict__ rank, RouteDev R,
                                                                 int* __restrict__ status) {
    __shared__ unsigned long long key[PM_DEVICE_PLAN_MAX_FRAMES];
    __shared__ int idx[PM_DEVICE_PLAN_MAX_FRAMES];
    __shared__ int size[PM_DEVICE_PLAN_MAX_FRAMES];
    __shared__ int partial[PLAN_THREADS];
    int np = 1;
    while (np < n_frames) np <<= 1;
    // ---- per frame: validate, count, key = its first seven ids (ascending, 9 bits each, high first)
    for (int f = threadIdx.x; f < np; f += PLAN_THREADS) {
        unsigned long long k = ~0ull;                 // padding sorts last
        int cnt = 0;
        if (f < n_frames) {
            const int lo = off[f], hi = off[f + 1];
            int n = hi - lo;
            if (lo < 0 || n < 0) { atomicCAS(status, 0, (int)PM_ERR_ARG); n = 0; }
            SetWalker w(ids + lo, n, max_adapters, rank);
            k = 0;
            for (int a = w.next(); a >= 0; a = w.next()) {
                if (cnt < 7) k |= (unsigned long long)(a + 1) << (9 * (6 - cnt));
                ++cnt;
            }
            if (cnt != n) atomicCAS(status, 0, (int)PM_ERR_ARG);       // invalid or repeated id
            if (cnt > max_set) { atomicCAS(status, 0, (int)PM_ERR_CAPACITY); cnt = max_set; }
        }
        key[f] = k; idx[f] = f; size[f] = cnt;
    }
    __syncthreads();
    // ---- bitonic sort by (key, frame index): equal sets end up adjacent, ties in caller order
    for (int k2 = 2; k2 <= np; k2 <<= 1) {
        for (int j = k2 >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < np; i += PLAN_THREADS) {
                const int p = i ^ j;
                if (p > i) {
                    const bool up = (i & k2) == 0;
                    const bool gt = key[i] > key[p] || (key[i] == key[p] && idx[i] > idx[p]);
                    if (gt == up) {
                        const unsigned long long tk = key[i]; key[i] = key[p]; key[p] = tk;
                        const int ti = idx[i]; idx[i] = idx[p]; idx[p] = ti;
                    }
                }
            }
            __syncthreads();
        }
    }
    // ---- slot CSR: exclusive scan of the sizes in slot order (each thread owns a contiguous chunk)
    const int per = (n_frames + PLAN_THREADS - 1) / PLAN_THREADS;
    const int lo = min(n_frames, (int)threadIdx.x * per), hi = min(n_frames, lo + per);
    int s = 0;
    for (int i = lo; i < hi; ++i) s += size[idx[i]];
    partial[threadIdx.x] = s;
    __syncthreads();
    for (int o = 1; o < PLAN_THREADS; o <<= 1) {
        const int v = (int)threadIdx.x >= o ? partial[threadIdx.x - o] : 0;
        __syncthreads();
        partial[threadIdx.x] += v;
        __syncthreads();
    }
    int run = partial[threadIdx.x] - s;
    if (threadIdx.x == 0) R.slot_off[0] = 0;
    for (int i = lo; i < hi; ++i) {
        const int f = idx[i];
        R.perm[i] = f;
        R.src_slot[i] = i;
        SetWalker w(ids + off[f], max(0, off[f + 1] - off[f]), max_adapters, rank);
        for (int j = 0; j < size[f]; ++j) R.slot_ids[run + j] = w.next();
        run += size[f];
        R.slot_off[i + 1] = run;
    }
}

// One block per pair of 128-row tiles: the union of the slabs its rows need (ascending), scales and
// per-half row masks.  Dynamic shared memory: bitmap over arena slabs, its word prefix, the list.
__global__ void __launch_bounds__(128) plan_tiles_kernel(int n_frames, int slabs_max, int max_adapters,
                                                         const int* __restrict__ rank,
                                                         const float* __restrict__ scale, RouteDev R,
                                                         int* __restrict__ status) {
    extern __shared__ int sm[];
    const int n_slabs = max_adapters * slabs_max;
    const int bw = (n_slabs + 31) / 32;
    unsigned int* bitmap = reinterpret_cast<unsigned int*>(sm);
    int* prefix = sm + bw;                      // [bw + 1]
    int* list = prefix + bw + 1;                // [slab_cap]
    const int T = R.tokens;
    const long long rows = (long long)n_frames * T;
    const long long r0 = (long long)blockIdx.x * 2 * PM_TILE_M, r1 = min(rows, r0 + 2 * PM_TILE_M);
    const int s_lo = (int)(r0 / T), s_hi = (int)((r1 - 1) / T);
    for (int w = threadIdx.x; w < bw; w += blockDim.x) bitmap[w] = 0u;
    __syncthreads();
    for (int slot = s_lo; slot <= s_hi; ++slot)
        for (int i = R.slot_off[slot] + threadIdx.x; i < R.slot_off[slot + 1]; i += blockDim.x) {
            const int a = R.slot_ids[i];
            const int ns = (rank[a] + PM_SLAB - 1) / PM_SLAB;
            for (int j = 0; j < ns; ++j) {
                const int b = a * slabs_max + j;
                atomicOr(&bitmap[b >> 5], 1u << (b & 31));
            }
        }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int w = 0; w < bw; ++w) { prefix[w] = run; run += __popc(bitmap[w]); }
        prefix[bw] = run;
        if (run > R.slab_cap) atomicCAS(status, 0, (int)PM_ERR_CAPACITY);
    }
    __syncthreads();
    const int count = min(prefix[bw], R.slab_cap);
    for (int w = threadIdx.x; w < bw; w += blockDim.x) {
        unsigned int bits = bitmap[w];
        int at = prefix[w];
        while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            if (at < R.slab_cap) list[at] = w * 32 + b;
            ++at;
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < count; i += blockDim.x) {
        const int slab = list[i], a = slab / slabs_max;
        uint32_t m[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int slot = s_lo; slot <= s_hi; ++slot) {
            bool member = false;
            for (int q = R.slot_off[slot]; q < R.slot_off[slot + 1]; ++q) member |= R.slot_ids[q] == a;
            if (!member) continue;
            const int a0 = (int)(max(r0, (long long)slot * T) - r0), a1 = (int)(min(r1, (long long)(slot + 1) * T) - r0);
            for (int r = a0; r < a1; ++r) m[r >> 5] |= 1u << (r & 31);
        }
        for (int half = 0; half < 2; ++half) {
            const size_t at = (size_t)(2 * blockIdx.x + half) * R.slab_cap + i;
            R.tile_slab[at] = slab;
            R.tile_scale[at] = scale[a];
            for (int q = 0; q < 4; ++q) R.tile_mask[at * 4 + q] = m[half * 4 + q];
        }
    }
    if (threadIdx.x == 0) {
        R.tile_nslabs[2 * blockIdx.x] = count;
        R.tile_nslabs[2 * blockIdx.x + 1] = count;
    }
}

}  // namespace

cudaError_t launch_device_plan(const Launch& L, const RouteDev& R, int n_frames, int max_set, int max_adapters,
                               int slabs_max, const int* off, const int* ids, const AdapterMeta& meta) {
    if (n_frames <= 0) return cudaSuccess;
    if (n_frames > PM_DEVICE_PLAN_MAX_FRAMES) return cudaErrorInvalidValue;
    ProfScope ps(L, KC_PLAN);
    plan_slots_kernel<<<1, PLAN_THREADS, 0, L.st>>>(n_frames, max_set, max_adapters, off, ids, meta.rank, R, L.status);
    BUMP(L);
    const long long rows = (long long)n_frames * R.tokens;
    const int n_pairs = (int)((rows + 2 * PM_TILE_M - 1) / (2 * PM_TILE_M));
    slabs_max = std::max(1, slabs_max);
    const int bw = (max_adapters * slabs_max + 31) / 32;
    const size_t smem = sizeof(int) * ((size_t)bw + bw + 1 + std::max(1, R.slab_cap));
    if (smem > 48 * 1024) return cudaErrorInvalidValue;
    plan_tiles_kernel<<<n_pairs, 128, smem, L.st>>>(n_frames, slabs_max, max_adapters, meta.rank,
                                                    meta.scale, R, L.status);
    BUMP(L);
    return cudaGetLastError();
}
