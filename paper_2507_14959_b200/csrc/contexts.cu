// Training-time context construction (Sec. 3.4, Algorithm 1) and its quality measure (Eq. 6).
//
// The label co-occurrence matrix is counted on the GPU from per-frame label bit sets (the format
// pm_select writes); the greedy construction itself is sequential over labels, works on a K x K
// matrix of at most a few hundred labels, and runs on the host.
#include <algorithm>
#include <numeric>
#include <vector>

#include "common.cuh"

namespace {

constexpr int COOC_MAX_LABELS_PER_FRAME = 64;

// One warp per frame: the set bits of its label words are listed in shared memory, then every
// ordered pair (diagonal included) adds 1 to co[i, j].  Counts stay exact in fp32 up to 2^24 frames.
__global__ void __launch_bounds__(256) cooccurrence_kernel(const uint32_t* __restrict__ labels, int n_frames,
                                                          int n_labels, float* __restrict__ co,
                                                          int* __restrict__ status) {
    __shared__ int ids[8][COOC_MAX_LABELS_PER_FRAME];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int f = blockIdx.x * 8 + warp;
    if (f >= n_frames) return;
    const int nw = (n_labels + 31) / 32;
    int n = 0;
    for (int w = 0; w < nw; ++w) {
        uint32_t word = labels[(size_t)f * nw + w];
        if (w == nw - 1 && (n_labels & 31)) word &= (1u << (n_labels & 31)) - 1u;
        const bool on = (word >> lane) & 1u;
        const int at = n + __popc(word & ((1u << lane) - 1u));
        if (on && at < COOC_MAX_LABELS_PER_FRAME) ids[warp][at] = w * 32 + lane;
        n += __popc(word);
    }
    if (n > COOC_MAX_LABELS_PER_FRAME) {             // more labels than a frame may carry here
        if (lane == 0 && status) atomicCAS(status, 0, (int)PM_ERR_CAPACITY);
        n = COOC_MAX_LABELS_PER_FRAME;
    }
    __syncwarp();
    for (int p = lane; p < n * n; p += 32) atomicAdd(&co[(size_t)ids[warp][p / n] * n_labels + ids[warp][p % n]], 1.0f);
}

}  // namespace

extern "C" {

int pm_cooccurrence(const uint32_t* labels, int n_frames, int n_labels, float* co, int32_t* status_out,
                    void* cuda_stream) {
    if (n_frames < 0 || n_labels <= 0 || !co || (n_frames > 0 && !labels)) return PM_ERR_ARG;
    if (n_frames > (1 << 24)) return PM_ERR_CAPACITY;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(co, 0, sizeof(float) * (size_t)n_labels * n_labels, st) != cudaSuccess) return PM_ERR_CUDA;
    if (status_out && cudaMemsetAsync(status_out, 0, sizeof(int32_t), st) != cudaSuccess) return PM_ERR_CUDA;
    if (n_frames == 0) return PM_OK;
    cooccurrence_kernel<<<(n_frames + 7) / 8, 256, 0, st>>>(labels, n_frames, n_labels, co, status_out);
    return cudaGetLastError() == cudaSuccess ? PM_OK : PM_ERR_CUDA;
}

int pm_build_contexts(const float* co, int n_labels, int max_size, int max_contexts, int allow_overlap,
                      int32_t* ctx_offsets, int32_t* ctx_ids, int* n_contexts) {
    if (!co || n_labels <= 0 || max_size <= 0 || max_contexts <= 0 || !ctx_offsets || !ctx_ids || !n_contexts)
        return PM_ERR_ARG;
    const int K = n_labels;
    auto C = [&](int i, int j) { return co[(size_t)i * K + j]; };
    std::vector<int> valid;
    for (int l = 0; l < K; ++l) if (C(l, l) > 0.f) valid.push_back(l);
    std::vector<int> order = valid;                   // most frequent first, ties by label
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return C(a, a) > C(b, b); });
    std::vector<std::vector<int>> ctx;
    std::vector<char> assigned(K, 0);
    std::vector<int> cand;
    for (int l : order) {
        if (!allow_overlap && assigned[l]) continue;
        cand.clear();
        for (int j : valid)
            if (j != l && C(l, j) > 0.f && (allow_overlap || !assigned[j])) cand.push_back(j);
        std::stable_sort(cand.begin(), cand.end(), [&](int a, int b) { return C(l, a) > C(l, b); });
        if ((int)cand.size() > max_size - 1) cand.resize(max_size - 1);
        cand.push_back(l);
        std::sort(cand.begin(), cand.end());
        if ((int)ctx.size() < max_contexts && std::find(ctx.begin(), ctx.end(), cand) == ctx.end()) {
            ctx.push_back(cand);
            if (!allow_overlap) for (int j : cand) assigned[j] = 1;
        }
    }
    std::vector<char> covered(K, 0);
    for (auto& c : ctx) for (int j : c) covered[j] = 1;
    for (int l : valid) {                             // leftovers go where they co-occur most, if there is room
        if (covered[l]) continue;
        int best = -1;
        double best_fit = -1.0;
        for (size_t c = 0; c < ctx.size(); ++c) {
            if ((int)ctx[c].size() >= max_size) continue;
            double fit = 0.0;
            for (int j : ctx[c]) fit += C(l, j);
            if (fit > best_fit) { best = (int)c; best_fit = fit; }
        }
        if (best >= 0) {
            ctx[best].insert(std::upper_bound(ctx[best].begin(), ctx[best].end(), l), l);
            covered[l] = 1;
        }
    }
    ctx_offsets[0] = 0;
    for (size_t c = 0; c < ctx.size(); ++c) {
        std::copy(ctx[c].begin(), ctx[c].end(), ctx_ids + ctx_offsets[c]);
        ctx_offsets[c + 1] = ctx_offsets[c] + (int)ctx[c].size();
    }
    *n_contexts = (int)ctx.size();
    return PM_OK;
}

int pm_intra_coherence(const float* co_norm, int n_labels, const int32_t* ctx_offsets, const int32_t* ctx_ids,
                       int n_contexts, double* out) {
    if (!co_norm || n_labels <= 0 || n_contexts < 0 || !out || (n_contexts > 0 && (!ctx_offsets || !ctx_ids)))
        return PM_ERR_ARG;
    double total = 0.0;
    for (int c = 0; c < n_contexts; ++c) {
        const int lo = ctx_offsets[c], hi = ctx_offsets[c + 1], n = hi - lo;
        if (n < 0) return PM_ERR_ARG;
        double s = 0.0;
        for (int a = lo; a < hi; ++a)
            for (int b = lo; b < hi; ++b) {
                const int i = ctx_ids[a], j = ctx_ids[b];
                if (i < 0 || i >= n_labels || j < 0 || j >= n_labels) return PM_ERR_ARG;
                if (a != b) s += co_norm[(size_t)i * n_labels + j];
            }
        if (n >= 2) total += s / ((double)n * (n - 1));
    }
    *out = n_contexts > 0 ? total / n_contexts : 0.0;
    return PM_OK;
}

}  // extern "C"
