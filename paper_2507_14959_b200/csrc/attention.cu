// Attention for the bf16 build.
#include "common.cuh"

cudaError_t launch_attention_mma(const Launch& L, const bf16* qkv, bf16* out, int n_frames, int tokens,
                                 int heads) {
    return launch_attention_simple<bf16>(L, qkv, out, n_frames, tokens, heads);
}
