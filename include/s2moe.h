/*
 * s2moe.h -- C ABI of the B200 (sm_100a) MoE verification layer with reuse-aware
 * expert gating (S2-MoE, Sec. 4.2) for self-speculative decoding.
 *
 * One call verifies one MoE layer for a whole batch or tree of B draft tokens:
 *
 *   1. router logits              l_{b,e} = h_b . W_r[e]
 *   2. reuse-aware expert gating  (Sec. 4.2, Eq. 4 and the two paragraphs after it)
 *        g_e      = sum_b w_b * l_{b,e}                    cross-token importance
 *        E*       = the `cap` experts with the largest g_e (ties: lower id)
 *        lambda_b = alpha * (l_(1) - l_(k+1))              top-1 minus (k+1)-th logit
 *        l'_{b,e} = l_{b,e} + lambda_b * [e in E*]         soft routing bias
 *        S_b      = the k experts with the largest l'_{b,e}
 *                   (ties: larger original logit, then lower id)
 *        p_{b,e}  = softmax over all E experts of l_b (weight_mode 0) or of l'_b
 *                   (weight_mode 1), taken at e in S_b, optionally renormalised
 *   3. union of the batch's choices and the number U of distinct experts
 *      (the quantity verification cost is proportional to: Sec. 3 "Challenge 2",
 *      Sec. 4.1 "Routing-aware Cost Estimation"); tokens bucketed by expert
 *   4. every distinct selected expert's SwiGLU FFN, its weights read from HBM once:
 *        y_b = sum_{e in S_b} p_{b,e} * W_d[e] ( silu(W_g[e] h_b) .* (W_u[e] h_b) )
 *            + sum_s c_b * FFN_shared_s(h_b),   c_b = sigmoid(h_b . w_sg) or 1
 *
 * The bias is off (standard top-k gating) when alpha == 0, cap >= n_experts or
 * top_k >= n_experts.  The tree structure of a draft tree is not an argument: the
 * layer treats tokens independently except through step 2, and ancestry enters only
 * through the confidences w_b, which the caller computes (Sec. 4.1, prefix
 * confidence p_i).
 *
 * Conventions
 *   - Every function returns S2MOE_OK (0) or a negative s2moe_status.  No exception
 *     crosses the boundary and there is no global state.
 *   - "dev" pointers are CUDA device memory owned by the caller; "host" pointers are
 *     ordinary host memory.  The library never frees or writes caller weights; it
 *     borrows the weight pointers for the lifetime of the context.
 *   - s2moe_verify_layer / s2moe_verify_stack are asynchronous on the given CUDA
 *     stream (a cudaStream_t passed as void*, NULL = legacy default stream), perform
 *     no host synchronisation and no allocation, and may be captured in a CUDA graph.
 *     Outputs are valid once the stream reaches that point.
 *   - A context may be used by one stream at a time (its workspace is shared by
 *     calls); it is bound to the device that was current in s2moe_create.
 *   - All device-side waits are bounded; a wait that gives up stores a non-zero code
 *     in a device status word that s2moe_last_device_status reads.
 *
 * Storage formats (s2moe_dtype)
 *   S2MOE_F32    IEEE binary32
 *   S2MOE_BF16   bfloat16
 *   S2MOE_Q4B32  symmetric block-int4: blocks of 32 weights along the contraction
 *                (last, contiguous) dimension; 16 bytes per block, weight i of the
 *                block in nibble i (byte i/2, low nibble for even i) stored as q+8
 *                with q in [-7,7]; one binary16 scale per block in a separate array;
 *                value = q * scale.  Weights only (not activations or the router).
 */
#ifndef S2MOE_H
#define S2MOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct s2moe_ctx s2moe_ctx;

typedef enum { S2MOE_F32 = 0, S2MOE_BF16 = 1, S2MOE_Q4B32 = 2 } s2moe_dtype;

typedef enum {
    S2MOE_OK = 0,
    S2MOE_EINVAL = -1,    /* bad config, shape, null pointer or alignment            */
    S2MOE_ERANGE = -2,    /* n_tokens > max_tokens, layer index out of range, more
                             active experts than an offloaded context has slots     */
    S2MOE_ENOMEM = -3,    /* workspace allocation failed                             */
    S2MOE_ECUDA = -4,     /* a CUDA call failed; see s2moe_last_cuda_error           */
    S2MOE_ETIMEOUT = -5   /* a bounded device-side wait gave up (device status != 0) */
} s2moe_status;

#define S2MOE_MAX_TOKENS 64      /* largest draft batch / tree per call       */
#define S2MOE_MAX_EXPERTS 256    /* largest number of routed experts          */
#define S2MOE_MAX_TOP_K 16

/* Weights of one layer.  All pointers dev, 16-byte aligned, row-major with the
 * contraction dimension contiguous. */
typedef struct {
    const void *router;    /* [E][d]      router_dtype                                      */
    const void *w_gate;    /* [E][f][d]   weight_dtype (Q4B32: [E][f][d/2] bytes)           */
    const void *w_up;      /* [E][f][d]                                                     */
    const void *w_down;    /* [E][d][f]   (Q4B32: [E][d][f/2] bytes)                        */
    const void *s_gate;    /* Q4B32 only: binary16 scales [E][f][d/32]; else NULL           */
    const void *s_up;      /*             [E][f][d/32]                                      */
    const void *s_down;    /*             [E][d][f/32]                                      */
    const void *sh_gate;   /* shared experts [n_sh][f_sh][d], NULL when n_shared == 0       */
    const void *sh_up;     /*                [n_sh][f_sh][d]                                */
    const void *sh_down;   /*                [n_sh][d][f_sh]                                */
    const void *sh_s_gate; /* Q4B32 scales of the shared experts, else NULL                 */
    const void *sh_s_up;
    const void *sh_s_down;
    const void *sh_scale;  /* [d] router_dtype: c_b = sigmoid(h_b . sh_scale); NULL: c_b = 1 */
} s2moe_layer_weights;

typedef struct {
    int32_t d_model;       /* d, multiple of 64                                             */
    int32_t d_ff;          /* f, multiple of 32                                             */
    int32_t n_experts;     /* E <= S2MOE_MAX_EXPERTS                                        */
    int32_t top_k;         /* 1 <= k <= min(E, S2MOE_MAX_TOP_K)                             */
    int32_t n_shared;      /* always-on shared experts (0..4)                               */
    int32_t d_ff_shared;   /* f_sh, multiple of 32 (ignored when n_shared == 0)             */
    int32_t act_dtype;     /* hidden states: S2MOE_F32 or S2MOE_BF16                        */
    int32_t router_dtype;  /* S2MOE_F32 or S2MOE_BF16                                       */
    int32_t weight_dtype;  /* expert weights: any s2moe_dtype                               */
    int32_t renorm;        /* 1: renormalise the k mixing weights of a token to sum 1       */
    int32_t cap;           /* |E*|, top_k <= cap <= E; cap == E turns the bias off          */
    float alpha;           /* lambda_b = alpha * (l_(1) - l_(k+1)); >= 0; 0: bias off       */
    int32_t weight_mode;   /* 0: mixing weights from l, 1: from l'                          */
    int32_t max_tokens;    /* 1..S2MOE_MAX_TOKENS: workspace bound for n_tokens             */
    int32_t n_layers;      /* >= 1                                                          */
    int32_t kernel_plan;   /* 0: automatic (plan 3 where it applies, else 2, else 1);
                              1: plain CUDA-core kernels (every format and batch size);
                              2: streaming mma.sync kernel (bf16 weights and activations);
                              3: streaming tcgen05 kernel: bf16 activations with bf16 weights
                                 (the kernel then starts while the gating still runs, on the
                                 shared experts and on every token's first expert by original
                                 logit, which stays selected for alpha < 1: Sec. 4.2; not for
                                 offloaded contexts), or with block-int4 weights when d_model, d_ff and
                                 d_ff_shared are multiples of 256 (the int4 values reach the
                                 tensor core as binary16 q * scale, rounded once: up to
                                 2^-12 relative per weight; block scales below 2^-17 lose
                                 precision in binary16's subnormal range; the hidden states
                                 are converted to binary16 for this kernel, so they must
                                 stay below 65504 in magnitude);
                              4: plan 3's kernel as the whole layer in ONE launch: its CTAs
                                 share the router's logit pass, meet once, every CTA runs the
                                 gating for itself, and the shared experts and the expert of
                                 every token's largest logit stream while it does (same
                                 formats as plan 3; not for offloaded contexts; needs room
                                 for n_tokens * n_experts float64 logits in shared memory).
                                 On demand only: measured slower than plan 3's two launches  */
} s2moe_config;

/*
 * Create a context for n_layers layers (problem statement of Sec. 4.2: the target
 * model's gating module and experts are given).  `layers` is a host array of
 * n_layers structs of dev pointers, copied by the call.  Allocates the workspace
 * (a few MB) on the current device; no weight is copied or repacked.
 * Errors: EINVAL (null, config out of the limits above, misaligned or missing
 * pointer), ENOMEM, ECUDA.  *out is NULL on error.
 */
int s2moe_create(const s2moe_config *config, const s2moe_layer_weights *layers, s2moe_ctx **out);

/*
 * Verify one layer for n_tokens draft tokens (steps 1-4 above; Sec. 4.2).
 *   hidden   dev [B][d] act_dtype, 16-byte aligned
 *   conf     dev [B] float w_b >= 0, or NULL for all ones (negative values: undefined)
 *   out      dev [B][d] float, overwritten with y
 *   sel_idx  dev [B][k] int32, experts of S_b in selection order (descending l')
 *   sel_w    dev [B][k] float, mixing weights p_{b,e} in the same order
 *   n_unique dev int32, U
 * n_tokens == 0 is a no-op returning S2MOE_OK.
 * Errors: EINVAL (null ctx/buffer, misaligned hidden/out), ERANGE (layer, n_tokens),
 * ECUDA (launch failure).
 */
int s2moe_verify_layer(s2moe_ctx *ctx, int32_t layer, int32_t n_tokens, const void *hidden,
                       const float *conf, float *out, int32_t *sel_idx, float *sel_w,
                       int32_t *n_unique, void *cuda_stream);

/*
 * Verify all n_layers layers back to back as independent layer problems: layer l reads
 * hidden + l*B*d elements (conf + l*B) and writes out + l*B*d, sel_idx + l*B*k,
 * sel_w + l*B*k and n_unique + l.  Same rules and errors as s2moe_verify_layer.
 */
int s2moe_verify_stack(s2moe_ctx *ctx, int32_t n_tokens, const void *hidden, const float *conf,
                       float *out, int32_t *sel_idx, float *sel_w, int32_t *n_unique,
                       void *cuda_stream);

/*
 * s2moe_verify_stack with HOST input and output buffers of the same shapes: copies
 * hidden (and conf, if not NULL) to staging memory the context owns, runs the stack,
 * copies out, sel_idx, sel_w and n_unique back and returns when all of it is complete.
 * The copies overlap the kernels: the inputs of the layers after the first and the outputs
 * of all layers but the last travel on two streams the context owns, ordered against
 * cuda_stream by events; sel_idx, sel_w and n_unique of all layers arrive in one copy in
 * page-locked memory of the context and are copied from there by the calling thread.  The host buffers must not be touched until the call returns;
 * page-locked host memory is needed for the overlap (pageable memory works, serialised).
 */
int s2moe_verify_stack_host(s2moe_ctx *ctx, int32_t n_tokens, const void *hidden_host,
                            const float *conf_host, float *out_host, int32_t *sel_idx_host,
                            float *sel_w_host, int32_t *n_unique_host, void *cuda_stream);

/* Free the workspace.  NULL is allowed.  The caller's buffers are untouched. */
int s2moe_destroy(s2moe_ctx *ctx);

/*
 * Expert-level offloading with hot experts kept resident (Sec. 5, "Edge memory constraints and
 * expert-level offloading": non-expert and shared parameters stay in device memory, individual
 * experts are fetched on demand, frequently activated experts are kept resident from an offline
 * profile).
 *
 * A context created by s2moe_create_offloaded keeps, per layer, a pool of n_slots device slots for
 * routed experts.  In its `layers`, w_gate, w_up, w_down and s_gate, s_up, s_down are HOST
 * pointers (page-locked memory recommended; same layouts as above, all n_experts experts);
 * router, the shared experts and sh_scale are dev pointers as usual.  The host arrays must stay
 * valid and unchanged for the life of the context.  pinned: host [n_layers][n_pinned] expert
 * ids that own slots 0..n_pinned-1 of their layer for good and are copied at create; NULL with
 * n_pinned == 0.  Replacement policy: see s2moe_cache_access.
 *
 * s2moe_verify_layer / _stack / _stack_host then work as before with two differences: between
 * the routing kernel and the expert kernel of a layer the call waits for the stream, reads the
 * active experts back and copies the missing ones into their slots (so the calls block and must
 * not be captured into a CUDA graph), and a step that activates more distinct experts than can
 * be resident at once fails with S2MOE_ERANGE.  Results are identical to those of a resident
 * context.  Needs the tcgen05 kernel (kernel_plan 0 or 3; bf16 activations; bf16 weights, or
 * block-int4 weights with d_model, d_ff, d_ff_shared multiples of 256) for every batch size up
 * to max_tokens: EINVAL otherwise.  Other errors: EINVAL (null, n_slots outside 1..n_experts,
 * n_pinned > n_slots, bad or repeated pinned id), ENOMEM, ECUDA.
 */
typedef struct {
    int32_t n_slots;        /* device slots per layer for routed experts               */
    int32_t n_pinned;       /* experts per layer that are never evicted (0..n_slots)    */
    const int32_t *pinned;  /* host [n_layers][n_pinned], or NULL                       */
} s2moe_residency;

int s2moe_create_offloaded(const s2moe_config *config, const s2moe_layer_weights *layers,
                           const s2moe_residency *residency, s2moe_ctx **out);

/* Totals over all layers since create: experts found resident, experts fetched, bytes copied
 * from host memory.  Any pointer may be NULL.  EINVAL when ctx is not offloaded. */
int s2moe_residency_stats(const s2moe_ctx *ctx, int64_t *hits, int64_t *misses, int64_t *bytes_fetched);

/* uses_out: host [n_experts], steps of `layer` that activated each expert since create: the
 * profile from which a hot set is chosen.  EINVAL, ERANGE (layer). */
int s2moe_residency_uses(const s2moe_ctx *ctx, int32_t layer, int64_t *uses_out);

/*
 * The replacement policy of one layer as a host-only object (no CUDA call): what an offloaded
 * context runs internally.  pinned experts own slots 0..n_pinned-1.  One access names n distinct
 * experts that must be resident together; slots_out[i] is the slot of experts[i], missed_out[i]
 * is 1 when it had to be fetched.  A missing expert takes the free slot of lowest index, else
 * the unpinned slot used least recently that is not wanted by this access (ties: lowest slot);
 * misses are served in the order given.  s2moe_cache_access returns ERANGE and changes nothing
 * when the experts cannot all be resident, an id is out of range or repeated.
 * All arrays host.
 */
typedef struct s2moe_cache s2moe_cache;
int s2moe_cache_create(int32_t n_experts, int32_t n_slots, const int32_t *pinned, int32_t n_pinned,
                       s2moe_cache **out);
int s2moe_cache_access(s2moe_cache *cache, const int32_t *experts, int32_t n, int32_t *slots_out,
                       int32_t *missed_out);
int s2moe_cache_destroy(s2moe_cache *cache);

/* Static description of a status code. */
const char *s2moe_strerror(int status);

/* Synchronises the device, stores the device status word (0 = no bounded wait gave
 * up) in *host_out and clears it.  Returns ETIMEOUT if it was non-zero. */
int s2moe_last_device_status(s2moe_ctx *ctx, int32_t *host_out);

/* The last cudaError_t a call on this context saw (0 = cudaSuccess). */
int s2moe_last_cuda_error(const s2moe_ctx *ctx);

/* The kernel plan a batch of n_tokens runs with (1, 2, 3 or 4; see s2moe_config.kernel_plan).
 * 0: NULL context, n_tokens out of range, or plan 2 / 3 was demanded and this batch size
 * does not fit its shared-memory layout (s2moe_verify_layer then returns EINVAL). */
int s2moe_kernel_plan(const s2moe_ctx *ctx, int32_t n_tokens);

/* Kernel launches issued through this context so far (not counting memsets/copies). */
int64_t s2moe_kernel_launches(const s2moe_ctx *ctx);

/* Unique-expert bytes a layer step reads for U distinct routed experts: expert weight
 * bytes (with Q4B32 scales) of U routed plus all shared experts. */
double s2moe_unique_expert_bytes(const s2moe_ctx *ctx, int32_t n_unique);

/*
 * Per-kernel timing for benchmarks.  Between s2moe_profile_begin and
 * s2moe_profile_end every kernel the context launches outside a graph capture is
 * bracketed by CUDA events on its launching stream (up to max_records launches;
 * later ones run untimed).  s2moe_profile_end synchronises the device and returns,
 * per kernel class c < n_classes, the summed duration in milliseconds and the
 * number of timed launches.  s2moe_kernel_class_name gives the kernel's name, or
 * NULL past the last class.  Do not use during stream capture.
 */
#define S2MOE_KERNEL_CLASSES 6
int s2moe_profile_begin(s2moe_ctx *ctx, int32_t max_records);
int s2moe_profile_end(s2moe_ctx *ctx, int32_t n_classes, double *ms_out, int64_t *launches_out);
const char *s2moe_kernel_class_name(int32_t cls);

/*
 * Diagnostics for tests: after synchronising, copy one workspace array of the LAST
 * verify call to host memory.  `what`:
 *   0 logits double [B][E]          1 counts  int32 [E + n_sh]   (tokens per expert)
 *   2 offsets int32 [E + n_sh + 1]  3 slot_token int32 [n_slots] 4 slot_w float [n_slots]
 *   5 active  int32 [n_active] (ids of experts with tokens, shared ones as E + s)
 *   6 header  int32 [4] = {n_active, n_slots, U, B}
 *   7 check   int32 [8]: first violation seen by a self-checking build of the kernels
 *             ({code, value, limit, block, ...}; all zero in the normal build)
 * n_slots = B*k + n_sh*B.  Returns EINVAL when `bytes` is smaller than the array.
 */
int s2moe_debug_read(s2moe_ctx *ctx, int32_t what, void *host_out, size_t bytes);

/*
 * Routing without any allocation (the paper has no counterpart; this is a convenience of
 * this library).  Some callers must not allocate device memory while they run: a serving
 * loop that has handed the whole device to its own memory pool, code that runs while a
 * framework's allocator is locked or a stream capture is open, or a latency-critical
 * path where a cudaMalloc (which may synchronise the device) is not acceptable.
 * s2moe_create allocates a workspace, so it is closed to them.  This entry point runs
 * steps 1-3 of the layer (router logits, reuse-aware gating, the unique-expert count)
 * with its scratch memory in a fixed array that is part of the library image: every GPU
 * that loads the library holds S2MOE_NOALLOC_SCRATCH_BYTES of it until the process exits.
 *
 *   cfg      the fields d_model, n_experts, top_k, act_dtype, router_dtype, renorm, cap,
 *            alpha and weight_mode are used, with the limits of s2moe_config; the rest
 *            is ignored
 *   router   dev [E][d] router_dtype          gate_vec  dev [d] router_dtype or NULL
 *   hidden   dev [B][d] act_dtype             conf      dev [B] float or NULL
 *   sel_idx  dev [B][k] int32, sel_w dev [B][k] float, n_unique dev int32: as in
 *            s2moe_verify_layer
 *   gate_out dev [B] float or NULL: sigmoid(h_b . gate_vec) when gate_vec is given
 *
 * Limits: n_tokens <= S2MOE_NOALLOC_MAX_TOKENS, n_experts <= S2MOE_NOALLOC_MAX_EXPERTS;
 * larger sizes return ERANGE and launch nothing.  The call is asynchronous on the stream
 * and calls no cudaMalloc, cudaFree or other allocating routine.  The first call on a
 * device looks up the scratch array's device address and raises the kernel's shared-memory
 * limit (once per device, with that device current); make that first call outside any
 * stream capture.  All calls on a device share the one scratch array: the call clears the
 * words that must start at zero, the rest keeps the previous call's contents, and two
 * calls that overlap on the GPU (different streams, no ordering between them) race.
 * Errors: EINVAL (null pointer, bad config, misaligned hidden or router), ERANGE, ECUDA.
 * The one bounded wait of the routing kernel reports through a status word inside the
 * scratch array, which every call clears: if that wait ever gives up, sel_idx, sel_w and
 * n_unique of that call stay unwritten although the call returned OK.  A caller that wants
 * to know reads the word with s2moe_route_noalloc_status before its next call.
 */
#define S2MOE_NOALLOC_MAX_TOKENS 64
#define S2MOE_NOALLOC_MAX_EXPERTS 128
#define S2MOE_NOALLOC_SCRATCH_BYTES (96 * 1024)
int s2moe_route_noalloc(const s2moe_config *cfg, int32_t n_tokens, const void *router, const void *gate_vec,
                        const void *hidden, const float *conf, int32_t *sel_idx, float *sel_w,
                        int32_t *n_unique, float *gate_out, void *cuda_stream);

/*
 * Device status of the last s2moe_route_noalloc call on the current device (no counterpart in
 * the paper).  Synchronises the device, copies the status word out of the scratch array (no
 * allocation) and returns OK with *host_out = 0, or ETIMEOUT with the device code when the
 * routing kernel's bounded wait gave up.  Before the first call on a device: OK and 0.
 */
int s2moe_route_noalloc_status(int32_t *host_out);

/*
 * Routing-aware adaptive speculative expansion (Sec. 4.1): the step that chooses which draft
 * candidates the verification layer will be run on.  Neither call uses a context, allocates
 * or synchronises; both are asynchronous on the given stream.
 *
 * s2moe_expert_masks -- predicted expert sets E_i as bit masks ("Routing-aware Cost
 * Estimation").  sel_idx: dev [n_tokens][top_k] expert ids (for example the sel_idx output of a
 * draft pass: s2moe_verify_layer on a context created with the draft top-k and alpha = 0).
 * masks: dev, word w of token t at masks[t * stride_words + w], bit (e % 64) of word (e / 64)
 * for expert e; ceil(n_experts / 64) words are written per token, so that the masks of several
 * layers can be interleaved by calling once per layer with an offset pointer.
 * Errors: EINVAL (null pointer, n_experts or top_k out of range, stride too small), ECUDA.
 */
int s2moe_expert_masks(const int32_t *sel_idx, int32_t n_tokens, int32_t top_k, int32_t n_experts,
                       uint64_t *masks, int32_t stride_words, void *cuda_stream);

/*
 * s2moe_adaptive_expand -- greedy admission by utility (Eq. 2, Eq. 3, "Adaptive Expansion").
 *   p_i   = product of p_tok along the path to candidate i            (prefix confidence)
 *   dC    = | E_i \ union of the admitted candidates' sets | * t_exp   (Eq. 2; the sets are given
 *           per MoE layer and the new experts of all layers are added up)
 *   U_i   = p_i * t_ar / (dC + c_draft[i])                            (Eq. 3; zero cost: +inf)
 * A candidate is eligible once its parent is admitted (parent -1: always).  Every step admits
 * the eligible candidate of largest utility (ties: lowest index) and stops when that utility is
 * below 1.  All of it in float64, one rounding per operation.
 *
 *   n_cand    1 .. S2MOE_EXPAND_MAX_CAND; parents must precede their children: a candidate
 *             whose parent index is not below its own is never admitted (nor is anything
 *             below it) and the call reports n_admitted = -1; the other outputs then hold
 *             the result for the well-formed rest
 *   parent    dev [n_cand]   index of the parent candidate, or -1
 *   p_tok     dev [n_cand]   token-level confidence of each candidate
 *   masks     dev [n_cand][n_layers][ceil(n_experts / 64)]   predicted expert sets
 *   c_draft   dev [n_cand]   draft expansion cost, or NULL for 0
 *   t_ar      latency of one autoregressive step of the target model; t_exp latency of one
 *             more expert in verification; both in the unit of c_draft
 *   admitted  dev [n_cand]   out: 1 / 0
 *   order     dev [n_cand]   out: admitted candidates in admission order, then -1
 *   n_admitted dev scalar    out: number of admitted candidates, or -1 (malformed parent[])
 *   union_out dev [n_layers][ceil(n_experts / 64)] or NULL   out: union of the admitted sets
 * Errors: EINVAL (null pointer, bad sizes), ERANGE (n_cand or n_layers * words beyond the
 * limits), ECUDA.
 */
#define S2MOE_EXPAND_MAX_CAND 256
#define S2MOE_EXPAND_MAX_WORDS 512      /* n_layers * ceil(n_experts / 64) */
int s2moe_adaptive_expand(int32_t n_cand, int32_t n_layers, int32_t n_experts, const int32_t *parent,
                          const float *p_tok, const uint64_t *masks, const float *c_draft, float t_ar,
                          float t_exp, int32_t *admitted, int32_t *order, int32_t *n_admitted,
                          uint64_t *union_out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* S2MOE_H */
