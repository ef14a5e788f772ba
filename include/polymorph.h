/*
 * polymorph.h -- C ABI of the B200 (sm_100a) Polymorph forward library.
 *
 * The library runs the data-parallel hot path of Polymorph (arXiv 2507.14959): the batched
 * forward pass of a shared ViT/DeiT backbone whose every linear layer computes
 *
 *        y = x W + b + sum_{a in S(frame)} s_a (x A_a) B_a            (Sec. 3.1)
 *
 * for each frame's own set S of active LoRA adapters (nothing is ever merged into W), followed by
 * the active adapters' class-subset heads, sigmoid scoring, the per-frame merge of the active
 * heads (Fig. 5b) and the greedy adapter-set (context) selection of Algorithm 2.
 *
 * Conventions
 *   - Every function returns PM_OK (0) or a negative pm_error; nothing aborts, nothing traps on
 *     the device.  pm_last_error() gives a text for the last failure on a handle.
 *   - "host" / "dev" in a comment says where a pointer must live.  All matrices are row-major;
 *     weights use the paper's row-vector convention W[in, out] (h = x W).
 *   - Ownership: pm_create / pm_register_adapter / pm_linear_* copy and convert what they are
 *     given (the caller may free it on return).  Frames, set lists, score and state buffers stay
 *     caller-owned and must outlive the stream work that uses them.
 *   - Work is enqueued on the given CUDA stream (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) and is asynchronous, except where a comment says it synchronises.
 *   - dtype 0: bf16 storage, fp32 accumulation, tensor-core kernels.  dtype 1: an all-fp32
 *     debug build of the same path on plain CUDA-core kernels.
 *   - Device-side waits are bounded; if one expires the kernel records PM_ERR_TIMEOUT in the
 *     handle's device status word (read it with pm_status) and returns normally.
 */
#ifndef POLYMORPH_H_
#define POLYMORPH_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PM_OK = 0,
    PM_ERR_ARG = -1,       /* NULL / out-of-range / malformed argument (e.g. non-monotone CSR)  */
    PM_ERR_STATE = -2,     /* adapter id not registered, cover table not built                  */
    PM_ERR_CAPACITY = -3,  /* more frames / adapters per frame / rank than the handle was sized  */
    PM_ERR_CUDA = -4,      /* a CUDA runtime or driver call failed                              */
    PM_ERR_TIMEOUT = -5,   /* a bounded device-side wait expired                                */
    PM_ERR_OOM = -6        /* device or host allocation failed                                  */
} pm_error;

typedef struct pm_handle_s* pm_handle;   /* opaque: owns every device copy of the model   */
typedef struct pm_linear_s* pm_linear;   /* opaque: one isolated base+multi-LoRA linear   */

/* Model geometry and capacities.  tokens = (img/patch)^2 + 1 (CLS first).  d / heads must be 64. */
typedef struct {
    int img, patch, d, layers, heads, mlp, n_classes;
    float ln_eps;
    int max_adapters;   /* adapter ids are in [0, max_adapters)                          */
    int max_rank;       /* largest LoRA rank that will be registered                     */
    int max_set;        /* largest |S| of a frame                                        */
    int max_frames;     /* largest batch passed to pm_forward / pm_select                */
    int dtype;          /* 0 = bf16 tensor-core build, 1 = fp32 debug build              */
} pm_config;

/* Backbone weights, host fp32.  Per-layer tensors are stacked on a leading [layers] axis. */
typedef struct {
    const float *patch_w;   /* [3*patch*patch, d], input order (channel, y, x)  */
    const float *patch_b;   /* [d]                                               */
    const float *cls;       /* [d]                                               */
    const float *pos;       /* [tokens, d]                                       */
    const float *ln1_g, *ln1_b;     /* [layers, d]                               */
    const float *qkv_w, *qkv_b;     /* [layers, d, 3d], [layers, 3d]; output columns [3][heads][64] */
    const float *proj_w, *proj_b;   /* [layers, d, d], [layers, d]               */
    const float *ln2_g, *ln2_b;     /* [layers, d]                               */
    const float *fc1_w, *fc1_b;     /* [layers, d, mlp], [layers, mlp]           */
    const float *fc2_w, *fc2_b;     /* [layers, mlp, d], [layers, d]             */
    const float *lnf_g, *lnf_b;     /* [d]                                       */
    const float *head_w, *head_b;   /* base head over all classes: [d, n_classes], [n_classes] */
} pm_backbone;

/* One LoRA adapter = one context C of the paper (Sec. 3.3): low-rank pairs for the adapted
 * linears, a head over its class subset, and its per-class accuracies a_{C,l} (Sec. 3.5). */
typedef struct {
    int rank;
    float scale;                 /* alpha / rank (Sec. 4: rank 16, alpha 32 -> 2)                  */
    const float* const* A;       /* host [layers*4] pointers, index l*4 + {0 qkv,1 proj,2 fc1,3 fc2}: */
    const float* const* B;       /*   A[in, rank], B[rank, out]; NULL pair = linear not adapted    */
    int n_cls;
    const int32_t* class_ids;    /* host [n_cls], distinct, each in [0, n_classes)                 */
    const float* head_w;         /* host [d, n_cls]                                                */
    const float* head_b;         /* host [n_cls]                                                   */
    const float* acc;            /* host [n_cls] accuracies a_{C,l}; NULL = all 1                  */
} pm_adapter;

/* ---- model lifetime -------------------------------------------------------------------- */

/* Builds the device model from host weights (ViT/DeiT encoder cited in Sec. 1; pre-LN blocks).
 * Allocates all activation and scratch memory for max_frames.  Synchronises the device. */
int pm_create(const pm_config* cfg, const pm_backbone* weights, pm_handle* out);

/* Registers (or replaces) adapter `adapter_id` (Sec. 3.1 low-rank pairs, Sec. 4 head).  The
 * handle's stream work must be idle.  Adapter ids order the tie-breaks of Algorithm 2. */
int pm_register_adapter(pm_handle h, int adapter_id, const pm_adapter* adapter);

/* Builds the class -> adapter cover tables used by pm_select from the registered adapters and
 * the accuracy threshold tau of Algorithm 2: for every class its first provider in Algorithm 2's
 * visiting order (fewest classes first, then lowest id) among adapters with a_{C,l} >= tau, and
 * the bit mask of all such providers.  Call after the last pm_register_adapter. */
int pm_set_cover(pm_handle h, float tau);

void pm_destroy(pm_handle h);

/* ---- the hot path ---------------------------------------------------------------------- */

/* Forward pass of n_frames frames (Sec. 3.1, Sec. 3.2, Fig. 5b).
 *   frames        dev, [n_frames, 3, img, img]; bf16 (dtype 0) or fp32 (dtype 1)
 *   set_offsets   host or dev int32 [n_frames+1], CSR over frames, set_offsets[0] = 0
 *   set_ids       host or dev int32 [set_offsets[n_frames]]: adapter ids, distinct per frame (any
 *                 order; they are applied in ascending id).  Device lists are copied to the host
 *                 first, which synchronises the stream.
 *   scores_out    dev fp32 [n_frames, n_classes]: sigmoid scores of the active adapters' heads,
 *                 scattered to class ids, maximum where several active adapters list a class,
 *                 0 for classes no active adapter lists
 *   base_out      dev fp32 [n_frames, n_classes] or NULL: sigmoid scores of the base head
 * Errors: PM_ERR_ARG (NULL, bad CSR, duplicate id), PM_ERR_STATE (unregistered id),
 * PM_ERR_CAPACITY (n_frames > max_frames, |S| > max_set).  No kernel is launched on error. */
int pm_forward(pm_handle h, const void* frames, int n_frames,
               const int32_t* set_offsets, const int32_t* set_ids,
               float* scores_out, float* base_out, void* cuda_stream);

/* The same forward in the per-branch arrangement of Fig. 2b / Fig. 5b (Sec. 3.1, Sec. 3.2): the
 * first trunk_layers blocks run once per frame without any adapter; from there the base model and
 * every active adapter continue as separate branches (one adapter alone per branch) through the
 * remaining blocks; each adapter's head reads its own branch, the base head reads the base branch,
 * and the branch outputs are merged as in pm_forward (maximum per class, 0 where no active adapter
 * lists the class).  Arguments as for pm_forward, plus
 *   trunk_layers  in [0, layers]: blocks shared by all branches.  No registered adapter may carry
 *                 A/B for a block below trunk_layers (the paper adapts the last 20 % of the blocks).
 *   base_out      dev fp32 [n_frames, n_classes] or NULL; with NULL no base branch is computed.
 * Capacity: n_frames + sum_f |S_f| branch slots when base_out is given, n_frames + sum_f max(|S_f|-1, 0)
 * without it; the total must not exceed max_frames.
 * Errors: as pm_forward, plus PM_ERR_STATE (an adapter touches a trunk block), PM_ERR_ARG
 * (trunk_layers out of range), PM_ERR_CAPACITY (too many branches).  No kernel is launched on error. */
int pm_forward_branched(pm_handle h, const void* frames, int n_frames,
                        const int32_t* set_offsets, const int32_t* set_ids, int trunk_layers,
                        float* scores_out, float* base_out, void* cuda_stream);

/* pm_forward for adapter sets that already live on the device, e.g. the lists pm_select wrote
 * (Algorithm 2 feeding the next frame, Sec. 3.2): the routing plan is built by kernels on the
 * stream, nothing is copied to the host and the stream is not synchronised, so forward -> select ->
 * forward runs without the host in between and the sequence can be recorded in a CUDA graph.
 *   set_offsets, set_ids   dev int32, as for pm_forward; they are read when the kernels run
 *   n_frames               at most PM_DEVICE_PLAN_MAX_FRAMES (and max_frames)
 * The lists cannot be checked on the host: an id that is out of range, not registered or repeated
 * is skipped, a frame with more than max_set ids keeps its max_set lowest, and the device status
 * word is set (PM_ERR_ARG / PM_ERR_CAPACITY, read with pm_status).  Frames are bucketed by their
 * first seven ids; results are the same as pm_forward's.
 * Errors: PM_ERR_ARG (NULL), PM_ERR_CAPACITY (n_frames).  No kernel is launched on error. */
#define PM_DEVICE_PLAN_MAX_FRAMES 2048
int pm_forward_device_sets(pm_handle h, const void* frames, int n_frames,
                           const int32_t* set_offsets, const int32_t* set_ids,
                           float* scores_out, float* base_out, void* cuda_stream);

/* Algorithm 2 (greedy context detection with conditional context copy) for n_frames streams.
 *   scores        dev fp32 [n_frames, n_classes]; Y_t = {k : scores[k] > score_thr}
 *   context_copy  Algorithm 2's flag
 *   has_prev      0: first frame of every stream (no Y_{t-1}, S_{t-1}: the greedy branch runs);
 *                 1: prev_labels / prev_offsets / prev_ids hold Y_{t-1} and S_{t-1}
 *   prev_labels   dev uint32 [n_frames, ceil(n_classes/32)] bit sets; read if has_prev, always
 *                 overwritten with Y_t; may be NULL only if has_prev == 0 (then nothing is kept)
 *   prev_offsets, prev_ids   dev int32 CSR of S_{t-1} (ascending ids); read only if has_prev
 *   next_offsets  dev int32 [n_frames+1]; next_ids dev int32 [ids_capacity]: CSR of S_t,
 *                 ascending ids.  If the result needs more than ids_capacity entries the lists are
 *                 truncated and PM_ERR_CAPACITY is recorded in the status word.
 * Needs pm_set_cover.  prev_* and next_* must not alias.  n_frames may differ from call to call.
 * An id in prev_ids outside [0, max_adapters), or a malformed prev_offsets pair, is skipped and
 * PM_ERR_ARG is recorded in the status word.  Calls on one handle share scratch memory: enqueue them
 * on one stream (or order them).
 * Every call also adds to the handle's stream-metric counters (see pm_metrics_read). */
int pm_select(pm_handle h, const float* scores, int n_frames, float score_thr, int context_copy,
              int has_prev, uint32_t* prev_labels,
              const int32_t* prev_offsets, const int32_t* prev_ids,
              int32_t* next_offsets, int32_t* next_ids, int ids_capacity, void* cuda_stream);

/* Selection for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a deployment variant of pm_select, same Algorithm 2 result.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a control loop with a
 * no-allocation rule after start-up, a plug-in that lives inside another framework's memory pool,
 * a process whose device memory has been handed out in full beforehand.  Such a caller cannot
 * build a pm_handle (pm_create / pm_set_cover allocate), so this call takes everything as plain
 * buffers and keeps its one piece of scratch -- the per-frame adapter bit masks between the two
 * phases of the kernel -- in a fixed array inside the library image:
 * PM_SELECT_STATIC_MAX_FRAMES x PM_SELECT_STATIC_MAX_ADAPTERS / 8 bytes = 128 KiB (plus a counter
 * word and a 256-byte status block), resident on every GPU that loads the library until the process exits.
 * The call itself performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 *   scores, prev_labels, prev_offsets, prev_ids, next_offsets, next_ids, ids_capacity,
 *   score_thr, context_copy, has_prev: exactly as in pm_select (all buffers dev)
 *   n_classes, n_adapters   sizes of the label space and of the adapter id range
 *   first      dev int32 [n_classes]: for each class the first adapter, in Algorithm 2's visiting
 *              order (fewest listed classes first, then lowest id), that lists it with accuracy
 *              >= tau; -1 if none
 *   provider   dev uint64 [n_classes, ceil(n_adapters/64)]: bit a of row k set iff adapter a lists
 *              class k with accuracy >= tau (the tables pm_set_cover builds inside a handle)
 *   status_out dev int32 or NULL: cleared by the call, then PM_ERR_CAPACITY is stored if the id list
 *              did not fit in ids_capacity (the lists are truncated), or PM_ERR_ARG if `first` or
 *              the previous lists hold an adapter id outside [0, n_adapters) or a malformed offset
 *              pair (such entries are skipped, nothing is read or written out of range because of
 *              them).  With NULL the conditions are not reported.
 * Errors: PM_ERR_ARG (NULL / non-positive sizes; a stream that belongs to another device than the
 * current one), PM_ERR_CAPACITY (n_frames > PM_SELECT_STATIC_MAX_FRAMES or n_adapters >
 * PM_SELECT_STATIC_MAX_ADAPTERS; nothing is launched), PM_ERR_CUDA.
 * Set-up: the first call on each device looks up the device address of the array (with that
 * device current -- make the stream's device current before calling).  Make that first call
 * before starting any stream capture.  Host threads may call concurrently (subject to the sharing
 * rule below); threads that race through a device's first call each do the look-up.
 * Sharing: all calls on a device use the same array and it keeps the previous call's contents.
 * The call clears the two words that must start at zero (status, block counter) on the stream; every
 * other word it reads it has written first.  Two calls whose kernels may overlap on the GPU --
 * different streams, no ordering -- race on the array: serialise them. */
#define PM_SELECT_STATIC_MAX_FRAMES 4096
#define PM_SELECT_STATIC_MAX_ADAPTERS 256
int pm_select_static(const float* scores, int n_frames, int n_classes, int n_adapters,
                     float score_thr, int context_copy, int has_prev, uint32_t* prev_labels,
                     const int32_t* prev_offsets, const int32_t* prev_ids,
                     const int32_t* first, const uint64_t* provider,
                     int32_t* next_offsets, int32_t* next_ids, int ids_capacity,
                     int32_t* status_out, void* cuda_stream);

/* Stream metrics of Sec. 3.4, counted on the device by pm_select over the sets it chooses:
 *   frames    number of (stream, step) selections made
 *   contexts  sum of |S_t| over them          -> AvgCoverage (Eq. 7) = contexts / frames
 *   switches  number of selections with has_prev whose S_t differs from S_{t-1}   (SwitchPenalty, Eq. 8)
 * pm_metrics_reset zeroes the counters on the stream; pm_metrics_read synchronises the stream and
 * copies them out (host pointers, each may be NULL).  Replayed CUDA graphs of pm_select count too. */
int pm_metrics_reset(pm_handle h, void* cuda_stream);
int pm_metrics_read(pm_handle h, void* cuda_stream, long long* frames, long long* contexts,
                    long long* switches);

/* Synchronises the stream and returns the device status word (PM_OK or the first recorded
 * error), then clears it. */
int pm_status(pm_handle h, void* cuda_stream);

const char* pm_last_error(pm_handle h);

/* Self-test of the bounded device-side waits (no counterpart in the paper: library diagnostics).
 * Launches one small CTA built from the same wait helper as the tensor-core kernels: one thread waits,
 * with a limit of limit_cycles GPU clock cycles (1 .. 1e8), on a barrier that is never signalled, the
 * other warps wait on a second such barrier with the library's own limit.  Expected outcome, read
 * after synchronising the stream: *status == PM_ERR_TIMEOUT (it is only written if it was 0),
 * trace[0] == 1 (the wait gave up), trace[1] == 3 (the other warps left through the abort flag),
 * trace[2] == 1 (tensor memory released).  Nothing faults and the context stays usable.
 *   status  dev int32, trace dev int32 [3] (cleared by the call). */
int pm_selftest_wait_timeout(long long limit_cycles, int32_t* status, int32_t* trace, void* cuda_stream);

/* The forward entry points record their launch sequence as a CUDA graph the second time they are
 * called with the same buffers, sizes and stream and the same widest adapter set, and replay it
 * from then on; the adapter sets themselves may change between replays (a new routing plan is
 * uploaded, or built by the recorded kernels for pm_forward_device_sets, before the replay reads it).  Not on the legacy default stream, not while the caller's stream is
 * itself being captured, not while pm_profile_enable is on.  pm_set_graphs(h, 0) switches this off
 * and frees the recorded graphs; default on. */
int pm_set_graphs(pm_handle h, int on);

/* Batches of a few frames of a small model (d <= 384 with 64-wide heads, mlp <= 1536, tokens <= 256,
 * max_set * ceil(max_rank / 16) <= 8, bf16 build, and n_frames * ceil(tokens / 16) <= the number of SMs) --
 * the single-stream operating point of Sec. 4 -- run the whole forward (patch embedding, every block with
 * its unmerged LoRA terms of Sec. 3.1, heads, sigmoid, merge) as ONE kernel in which a CTA owns 16 token
 * rows from the first layer to the last.  pm_forward and pm_forward_device_sets use it for such batches
 * (same results within rounding as the layer-by-layer kernels; about 330 against 545 us per DeiT-tiny
 * frame and step on a B200); pm_set_small_batch_kernel(h, 0) sends them through the layer-by-layer kernels
 * instead.  Default on. */
int pm_set_small_batch_kernel(pm_handle h, int on);

/* Number of kernels the library has launched on this handle since creation (kernels of a replayed graph included). */
long long pm_launch_count(pm_handle h);

/* Device timing of the library's own kernels, by class, with CUDA events recorded on the launching
 * stream around each launch site: class 0 fused base+LoRA GEMM (patch embed included), 1 LoRA
 * shrink, 2 attention, 3 LayerNorm / row statistics, 4 patch gather, CLS rows and branch fan-out,
 * 5 final LayerNorm + heads + sigmoid + merge, 6 Algorithm 2 selection, 7 routing plan built on the
 * device.  pm_profile_enable(h, 1) clears and starts recording, (h, 0) stops.  pm_profile_read
 * synchronises the stream, returns total milliseconds and launch-site counts per class (arrays of
 * PM_PROFILE_CLASSES) since the last read, and clears them. */
#define PM_PROFILE_CLASSES 8
int pm_profile_enable(pm_handle h, int on);
int pm_profile_read(pm_handle h, void* cuda_stream, double* ms_by_class, long long* launches_by_class);

/* Host-side cost of the routing plan (Sec. 3.2: frames are bucketed by adapter set before the fused
 * linears run): number of plans pm_forward / pm_forward_branched have built on the host since the
 * handle was created (a call whose sets equal the previous call's reuses the uploaded plan and builds
 * nothing) and the total host time spent building them, in milliseconds.  Either pointer may be NULL. */
int pm_plan_stats(pm_handle h, long long* plans_built, double* host_ms);

/* ---- training-time context construction (Sec. 3.4) -------------------------------------- */

/* Label co-occurrence counts from per-frame label bit sets (the layout pm_select keeps in
 * prev_labels): co[i, j] = number of frames whose set holds both i and j; co[i, i] = frames holding i.
 *   labels      dev uint32 [n_frames, ceil(n_labels/32)], bit k%32 of word k/32 = label k
 *   co          dev fp32 [n_labels, n_labels], overwritten (counts are exact: n_frames <= 2^24)
 *   status_out  dev int32 or NULL: PM_ERR_CAPACITY if a frame carries more than 64 labels (its first
 *               64 are counted)
 * Asynchronous on the stream.  Errors: PM_ERR_ARG, PM_ERR_CAPACITY (n_frames), PM_ERR_CUDA. */
int pm_cooccurrence(const uint32_t* labels, int n_frames, int n_labels, float* co,
                    int32_t* status_out, void* cuda_stream);

/* Algorithm 1 (BuildContexts).  Host function, host pointers.
 *   co             host fp32 [n_labels, n_labels] co-occurrence (symmetric; diagonal = label frequency)
 *   max_size       B: no context holds more labels; max_contexts: M_max; allow_overlap: the flag
 *   ctx_offsets    host int32 [max_contexts + 1], ctx_ids host int32 [max_contexts * max_size]: the
 *                  contexts as CSR of ascending label ids, in creation order; *n_contexts their number
 * Valid labels (co[l, l] > 0) are visited from the most to the least frequent (ties: lower label);
 * a cluster is the label plus its up to B-1 strongest co-occurring valid neighbours (co > 0; ties:
 * lower label; without overlap only unassigned ones); a cluster equal to a kept context is dropped;
 * labels left uncovered go, in ascending order, to the context with room whose members co-occur
 * with them most (ties: earlier context), or stay uncovered if none has room. */
int pm_build_contexts(const float* co, int n_labels, int max_size, int max_contexts, int allow_overlap,
                      int32_t* ctx_offsets, int32_t* ctx_ids, int* n_contexts);

/* IntraCoherence (Eq. 6) of a context set under a normalised co-occurrence matrix (host pointers):
 * mean over contexts of the mean co_norm[i, j] over ordered pairs i != j; single-label contexts
 * contribute 0. */
int pm_intra_coherence(const float* co_norm, int n_labels, const int32_t* ctx_offsets,
                       const int32_t* ctx_ids, int n_contexts, double* out);

/* ---- single operators (the same kernels pm_forward uses), for unit tests and sweeps ----- */

/* One base + multi-LoRA linear y = epilogue(x W + b + sum_a s_a (x A_a) B_a)   (Sec. 3.1).
 *   w host fp32 [k_in, n_out]; bias host fp32 [n_out]
 *   epilogue 0: none, 1: exact-erf GELU, 2: y += residual
 * k_in and n_out must be multiples of 64. */
int pm_linear_create(int k_in, int n_out, const float* w, const float* bias,
                     int max_adapters, int max_rank, int max_set, int max_frames, int tokens,
                     int epilogue, int dtype, pm_linear* out);
/* A host fp32 [k_in, rank], B host fp32 [rank, n_out]. */
int pm_linear_register(pm_linear lin, int adapter_id, int rank, float scale,
                       const float* A, const float* B);
/* x dev [n_frames*tokens, k_in], residual dev [n_frames*tokens, n_out] or NULL (epilogue 2 only),
 * y dev [n_frames*tokens, n_out]; element type per dtype.  set_offsets / set_ids: host CSR. */
int pm_linear_forward(pm_linear lin, const void* x, int n_frames,
                      const int32_t* set_offsets, const int32_t* set_ids,
                      const void* residual, void* y, void* cuda_stream);
int pm_linear_status(pm_linear lin, void* cuda_stream);
const char* pm_linear_last_error(pm_linear lin);
void pm_linear_destroy(pm_linear lin);

/* Row-wise LayerNorm of x[rows, d] (biased variance, fp32 statistics); gamma/beta dev fp32 [d].
 * d must be a multiple of 8 and at most 1024. */
int pm_layernorm(const void* x, const float* gamma, const float* beta, void* y,
                 int rows, int d, float eps, int dtype, void* cuda_stream);

/* softmax(q k^T / 8) v per (frame, head), head dim 64; qkv dev [n_frames*tokens, 3*heads*64]
 * with columns ordered [3][heads][64]; out dev [n_frames*tokens, heads*64]. */
int pm_attention(const void* qkv, void* out, int n_frames, int tokens, int heads, int dtype,
                 void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* POLYMORPH_H_ */
