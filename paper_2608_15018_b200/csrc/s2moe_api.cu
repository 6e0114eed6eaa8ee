// C ABI of the MoE verification library: context, validation, kernel dispatch.
// See include/s2moe.h for the contract of every entry point.
#include "../../include/s2moe.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "ffn_simple.cuh"
#include "ffn_stream.cuh"
#include "expand.cuh"
#include "ffn_tc.cuh"
#include "route.cuh"
#include "layer_tc.cuh"

#include "expert_cache.h"

using namespace s2moe;

struct s2moe_ctx {
    s2moe_config cfg;
    Shape shape;
    std::vector<LayerPtrs> layers;
    Workspace ws;
    void *slab = nullptr;          // one allocation behind ws
    size_t slab_bytes = 0;
    // staging for the host-buffer entry point
    void *st_hidden = nullptr;
    float *st_conf = nullptr, *st_out = nullptr, *st_selw = nullptr;
    int32_t *st_sel = nullptr, *st_nu = nullptr;
    int device = 0;
    int plan = 1;
    int n_sm = 0;
    __nv_bfloat16 *act_hi = nullptr, *act_lo = nullptr;
    size_t act_elems = 0;
    cudaLaunchAttribute pdl_attr{};
    bool use_pdl = true;                  // S2MOE_NO_PDL=1 in the environment turns it off
    bool pdl_in_graph = false;            // S2MOE_PDL_IN_GRAPH=1: also under stream capture
    void *hperm = nullptr;                // int4 plan 3: column-permuted copy of the hidden states
    double *lpart = nullptr;              // partial router logits [piece][token][row] (logit pass by warp tasks)
    int route_task_from = 48;             // batches of this many tokens and more take the logit pass by warp tasks
    bool early_start = true;              // bf16 tensor-core plan: the expert kernel starts under the gating (S2MOE_NO_EARLY=1: off)
    int wave_split[2] = {0, 16};          // S2MOE_WAVES=a,b: where waves 1 and 2 of the bf16 expert kernel begin (16ths; 0: the built-in)
    int bf16_kg2_from = 2;                // batches of this many tokens and more: two k-tiles per ring stage (bf16)
    float *pre = nullptr;                 // plan 3: fp32 pre-activations [gate|up][slot][f]
    std::vector<TcMaps> tc_maps;          // plan 3: per layer, weight maps filled at create
    void *encode_tiled = nullptr;         // cuTensorMapEncodeTiled, looked up through the runtime
    int last_cuda = 0;
    int64_t launches = 0;
    int last_B = 0;
    // optional per-kernel timing (CUDA events on the launching stream)
    bool prof_on = false;
    std::vector<cudaEvent_t> prof_ev;   // 2 per record
    std::vector<int> prof_cls;
    size_t prof_cap = 0;
    // expert offloading (s2moe_create_offloaded): the routed experts' weights live in host memory,
    // n_w_experts = n_slots of them at a time in a device pool that the weight pointers of
    // `layers` point into
    bool offload = false;
    int n_w_experts = 0;                  // experts the device weight tensors hold (n_experts, or n_slots)
    std::vector<ExpertCache> caches;      // per layer
    std::vector<LayerPtrs> host_w;        // per layer: host pointers of the routed experts
    void *pool = nullptr;
    int32_t *h_route = nullptr;           // pinned: {n_active, n_slots, U, B} and the active list
    int32_t *h_slot_of = nullptr;         // pinned [E]
    int32_t *d_slot_of = nullptr;         // device [E]
    size_t mat_bytes[6] = {0, 0, 0, 0, 0, 0};   // one expert's bytes in w_gate, w_up, w_down, s_gate, s_up, s_down
    int64_t fetched_bytes = 0;
    // host-buffer entry point: streams and events of its copies, made at the first call
    cudaStream_t cs_in = nullptr, cs_out = nullptr;
    cudaEvent_t ev_copy[4] = {nullptr, nullptr, nullptr, nullptr};
    uint8_t *h_small = nullptr;           // page-locked landing place of the indices, weights and counts
};

struct s2moe_cache {
    ExpertCache c;
};

enum KernelClass { KC_ROUTER = 0, KC_GATING = 1, KC_GATEUP = 2, KC_DOWN = 3, KC_STREAM = 4, KC_TC = 5, KC_LAYER = 6, KC_COUNT = 7 };

namespace {

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(s2moe_ctx *ctx, cudaError_t e)
{
    if (ctx) ctx->last_cuda = (int)e;
    return S2MOE_ECUDA;
}

#define CU(ctx, call)                                       \
    do {                                                    \
        cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return cuda_fail((ctx), e_); \
    } while (0)

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Brackets one kernel launch: counts it and, when timing is on, records an event
// before and after it on the launching stream.
struct LaunchScope {
    s2moe_ctx *ctx;
    cudaStream_t st;
    long rec = -1;
    LaunchScope(s2moe_ctx *c, int cls, cudaStream_t s) : ctx(c), st(s)
    {
        ctx->launches++;
        if (ctx->prof_on && ctx->prof_cls.size() < ctx->prof_cap) {
            rec = (long)ctx->prof_cls.size();
            ctx->prof_cls.push_back(cls);
            cudaEventRecord(ctx->prof_ev[2 * rec], st);
        }
    }
    ~LaunchScope()
    {
        if (rec >= 0) cudaEventRecord(ctx->prof_ev[2 * rec + 1], st);
    }
};

int validate_config(const s2moe_config *c)
{
    if (!c) return S2MOE_EINVAL;
    if (c->d_model < 64 || c->d_model % 64) return S2MOE_EINVAL;
    if (c->d_ff < 32 || c->d_ff % 32) return S2MOE_EINVAL;
    if (c->n_experts < 1 || c->n_experts > S2MOE_MAX_EXPERTS) return S2MOE_EINVAL;
    if (c->top_k < 1 || c->top_k > c->n_experts || c->top_k > S2MOE_MAX_TOP_K) return S2MOE_EINVAL;
    if (c->n_shared < 0 || c->n_shared > kMaxShared) return S2MOE_EINVAL;
    if (c->n_shared > 0 && (c->d_ff_shared < 32 || c->d_ff_shared % 32)) return S2MOE_EINVAL;
    if (c->act_dtype != S2MOE_F32 && c->act_dtype != S2MOE_BF16) return S2MOE_EINVAL;
    if (c->router_dtype != S2MOE_F32 && c->router_dtype != S2MOE_BF16) return S2MOE_EINVAL;
    if (c->weight_dtype < S2MOE_F32 || c->weight_dtype > S2MOE_Q4B32) return S2MOE_EINVAL;
    if (c->renorm != 0 && c->renorm != 1) return S2MOE_EINVAL;
    if (c->cap < c->top_k || c->cap > c->n_experts) return S2MOE_EINVAL;
    if (!(c->alpha >= 0.0f)) return S2MOE_EINVAL;
    if (c->weight_mode != 0 && c->weight_mode != 1) return S2MOE_EINVAL;
    if (c->max_tokens < 1 || c->max_tokens > S2MOE_MAX_TOKENS) return S2MOE_EINVAL;
    if (c->n_layers < 1) return S2MOE_EINVAL;
    if (c->kernel_plan < 0 || c->kernel_plan > 4) return S2MOE_EINVAL;
    // the tcgen05 plan covers bf16 activations with bf16 or block-int4 weights
    if (c->kernel_plan >= 3 && (c->weight_dtype == S2MOE_F32 || c->act_dtype != S2MOE_BF16)) return S2MOE_EINVAL;
    // the mma.sync plan covers bf16 weights with bf16 activations
    if (c->kernel_plan == 2 && (c->weight_dtype != S2MOE_BF16 || c->act_dtype != S2MOE_BF16)) return S2MOE_EINVAL;
    return S2MOE_OK;
}

int validate_layer(const s2moe_config *c, const s2moe_layer_weights *w)
{
    const void *need[] = {w->router, w->w_gate, w->w_up, w->w_down};
    for (const void *p : need)
        if (!p || !aligned16(p)) return S2MOE_EINVAL;
    if (c->weight_dtype == S2MOE_Q4B32) {
        const void *sc[] = {w->s_gate, w->s_up, w->s_down};
        for (const void *p : sc)
            if (!p || !aligned16(p)) return S2MOE_EINVAL;
    }
    if (c->n_shared > 0) {
        const void *shp[] = {w->sh_gate, w->sh_up, w->sh_down};
        for (const void *p : shp)
            if (!p || !aligned16(p)) return S2MOE_EINVAL;
        if (c->weight_dtype == S2MOE_Q4B32) {
            const void *sc[] = {w->sh_s_gate, w->sh_s_up, w->sh_s_down};
            for (const void *p : sc)
                if (!p || !aligned16(p)) return S2MOE_EINVAL;
        }
        if (w->sh_scale && !aligned16(w->sh_scale)) return S2MOE_EINVAL;
    }
    return S2MOE_OK;
}

// ---- dispatch over storage formats ------------------------------------------

// Launch configuration with programmatic stream serialization: the kernel may start before
// the one in front of it in the stream has finished; it calls griddepcontrol.wait before it
// touches anything that kernel writes.  Only kernels that contain that wait are launched so.
cudaLaunchConfig_t pdl_config(s2moe_ctx *ctx, int grid, int block, size_t smem, cudaStream_t st, bool in_graph = false)
{
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)grid);
    lc.blockDim = dim3((unsigned)block);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    ctx->pdl_attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    // measured: plain stream launches gain about 4 % from it, a captured graph loses about 1 %
    // (its kernel nodes already follow each other closely), so it is left out under capture unless
    // the kernel does real work before its wait (in_graph: the expert kernel that starts under the
    // gating, and the routing kernel in front of it)
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    const bool capturing = cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap != cudaStreamCaptureStatusNone;
    ctx->pdl_attr.val.programmaticStreamSerializationAllowed = (ctx->use_pdl && (!capturing || ctx->pdl_in_graph || in_graph)) ? 1 : 0;
    lc.attrs = &ctx->pdl_attr;
    lc.numAttrs = 1;
    return lc;
}

size_t route_smem(int B, int E)
{
    const size_t a = (size_t)B * E + (size_t)B, b = (size_t)(kRouteThreads / 32) * kRouteTok;
    return sizeof(double) * (a > b ? a : b);
}

template <int ACT, int RT>
void launch_route_t(s2moe_ctx *ctx, const Shape &sh, const LayerPtrs &lp, int B, const void *hidden, const float *conf,
                    int32_t *sel_idx, float *sel_w, int32_t *n_unique, const ZeroList &zl, cudaStream_t st)
{
    // one block per router row; more (up to one per SM) when there is a lot to clear or copy:
    // 16 bytes per thread and pass, a handful of passes at most
    const int rows = sh.E + (lp.sh_scale ? 1 : 0);
    const unsigned long long units = zl.n16[0] + zl.n16[1] + zl.n16[2] + zl.perm_n16;
    // batches of more than 4 tokens: their tokens in groups of at least 4, each group with its own
    // set of row blocks, as many sets as run beside each other (a block per SM); measured at 64
    // experts: 1.1 % of a layer at B = 8, 4.5 % at B = 16
    ZeroList zg = zl;
    zg.groups = 1;
    zg.ksplit = 0;
    zg.lpart = nullptr;
    int grid;
    const int task_from = ctx->route_task_from;
    if (ctx->lpart && B >= task_from) {
        // the logit pass as warp tasks: pieces of the contraction so that the warps of a full grid
        // have about one task each
        const int tgs = (B + 7) / 8, warps = ctx->n_sm * (kRouteThreadsBig / 32);
        int ks = warps / (rows * tgs);
        if (ks > 8) ks = 8;
        if (ks > sh.d / 128) ks = sh.d / 128;
        zg.ksplit = ks < 1 ? 1 : ks;
        zg.lpart = ctx->lpart;
        const int tasks = rows * tgs * zg.ksplit, blocks = (tasks + kRouteThreadsBig / 32 - 1) / (kRouteThreadsBig / 32);
        grid = blocks < ctx->n_sm ? blocks : ctx->n_sm;
        // more blocks (up to one per SM) when there is a lot to clear or copy
        const unsigned long long want = (units + kRouteThreadsBig * 4 - 1) / (kRouteThreadsBig * 4);
        if (want > (unsigned long long)grid) grid = (int)(want > (unsigned long long)ctx->n_sm ? (unsigned long long)ctx->n_sm : want);
    } else {
    if (B > 4) {
        const int fit = ctx->n_sm / rows, want = (B + 3) / 4;
        zg.groups = fit < 1 ? 1 : (want < fit ? want : fit);
    }
    grid = rows * zg.groups;
    if (units > (unsigned long long)rows * kRouteThreads * 4) {
        const unsigned long long want = (units + kRouteThreads * 4 - 1) / (kRouteThreads * 4);
        grid = (int)(want > (unsigned long long)ctx->n_sm ? (unsigned long long)ctx->n_sm : want);
        if (grid < rows * zg.groups) grid = rows * zg.groups;
    }
    }
    LaunchScope scope(ctx, KC_ROUTER, st);
    if (zg.ksplit > 0) {
        cudaLaunchConfig_t lc = pdl_config(ctx, grid, kRouteThreadsBig, route_smem(B, sh.E), st, zl.early != 0);
        if (sh.E <= 64)
            cudaLaunchKernelEx(&lc, route_kernel_big<ACT, RT, 2>, sh, B, ctx->ws, hidden, (const void *)lp.router,
                               (const void *)lp.sh_scale, conf, sel_idx, sel_w, n_unique, zg);
        else if (sh.E <= 128)
            cudaLaunchKernelEx(&lc, route_kernel_big<ACT, RT, 4>, sh, B, ctx->ws, hidden, (const void *)lp.router,
                               (const void *)lp.sh_scale, conf, sel_idx, sel_w, n_unique, zg);
        else
            cudaLaunchKernelEx(&lc, route_kernel_big<ACT, RT, 8>, sh, B, ctx->ws, hidden, (const void *)lp.router,
                               (const void *)lp.sh_scale, conf, sel_idx, sel_w, n_unique, zg);
        return;
    }
    cudaLaunchConfig_t lc = pdl_config(ctx, grid, kRouteThreads, route_smem(B, sh.E), st, zl.early != 0);
    if (sh.E <= 64)
        cudaLaunchKernelEx(&lc, route_kernel<ACT, RT, 2>, sh, B, ctx->ws, hidden, (const void *)lp.router,
                           (const void *)lp.sh_scale, conf, sel_idx, sel_w, n_unique, zg);
    else if (sh.E <= 128)
        cudaLaunchKernelEx(&lc, route_kernel<ACT, RT, 4>, sh, B, ctx->ws, hidden, (const void *)lp.router,
                           (const void *)lp.sh_scale, conf, sel_idx, sel_w, n_unique, zg);
    else
        cudaLaunchKernelEx(&lc, route_kernel<ACT, RT, 8>, sh, B, ctx->ws, hidden, (const void *)lp.router,
                           (const void *)lp.sh_scale, conf, sel_idx, sel_w, n_unique, zg);
}

void launch_route(s2moe_ctx *ctx, const Shape &sh, const LayerPtrs &lp, int B, const void *hidden, const float *conf,
                  int32_t *sel_idx, float *sel_w, int32_t *n_unique, const ZeroList &zl, cudaStream_t st)
{
    const bool af = sh.act_dtype == DT_F32, rf = sh.router_dtype == DT_F32;
    if (af && rf) launch_route_t<DT_F32, DT_F32>(ctx, sh, lp, B, hidden, conf, sel_idx, sel_w, n_unique, zl, st);
    else if (af) launch_route_t<DT_F32, DT_BF16>(ctx, sh, lp, B, hidden, conf, sel_idx, sel_w, n_unique, zl, st);
    else if (rf) launch_route_t<DT_BF16, DT_F32>(ctx, sh, lp, B, hidden, conf, sel_idx, sel_w, n_unique, zl, st);
    else launch_route_t<DT_BF16, DT_BF16>(ctx, sh, lp, B, hidden, conf, sel_idx, sel_w, n_unique, zl, st);
}

template <int ACT, int RT>
cudaError_t prepare_route_t(int bytes)
{
    cudaError_t e = cudaFuncSetAttribute(route_kernel<ACT, RT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(route_kernel<ACT, RT, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(route_kernel<ACT, RT, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(route_kernel_big<ACT, RT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(route_kernel_big<ACT, RT, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(route_kernel_big<ACT, RT, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e;
}

cudaError_t prepare_route()
{
    const int bytes = (int)route_smem(kMaxTokens, kMaxExperts);
    cudaError_t e = prepare_route_t<DT_F32, DT_F32>(bytes);
    if (e == cudaSuccess) e = prepare_route_t<DT_F32, DT_BF16>(bytes);
    if (e == cudaSuccess) e = prepare_route_t<DT_BF16, DT_F32>(bytes);
    if (e == cudaSuccess) e = prepare_route_t<DT_BF16, DT_BF16>(bytes);
    return e;
}

constexpr size_t kSimpleSmem = (size_t)kSimpleTokChunk * kSimpleKChunk * sizeof(float);

template <int WT, int ACT>
void launch_simple(s2moe_ctx *ctx, const LayerPtrs &lp, const void *hidden, float *out, cudaStream_t st)
{
    const Shape &sh = ctx->shape;
    const int groups = sh.E + sh.n_sh;
    const int fmax = sh.n_sh > 0 && sh.f_sh > sh.f ? sh.f_sh : sh.f;
    const dim3 block(kSimpleWarps * 32);
    const dim3 g1((fmax + kSimpleWarps - 1) / kSimpleWarps, groups);
    const dim3 g2((sh.d + kSimpleWarps - 1) / kSimpleWarps, groups);
    {
        LaunchScope scope(ctx, KC_GATEUP, st);
        ffn_gateup_simple<WT, ACT><<<g1, block, kSimpleSmem, st>>>(sh, lp, ctx->ws, hidden);
    }
    {
        LaunchScope scope(ctx, KC_DOWN, st);
        ffn_down_simple<WT><<<g2, block, kSimpleSmem, st>>>(sh, lp, ctx->ws, out);
    }
}

template <int WT, int ACT>
cudaError_t prepare_simple()
{
    cudaError_t e = cudaFuncSetAttribute(ffn_gateup_simple<WT, ACT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kSimpleSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(ffn_down_simple<WT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSimpleSmem);
}

#define DISPATCH_WT_ACT(ctx, FN, ...)                                                    \
    do {                                                                                 \
        const int wt_ = (ctx)->shape.weight_dtype, at_ = (ctx)->shape.act_dtype;         \
        if (wt_ == DT_F32 && at_ == DT_F32) FN<DT_F32, DT_F32>(__VA_ARGS__);             \
        else if (wt_ == DT_F32) FN<DT_F32, DT_BF16>(__VA_ARGS__);                        \
        else if (wt_ == DT_BF16 && at_ == DT_F32) FN<DT_BF16, DT_F32>(__VA_ARGS__);      \
        else if (wt_ == DT_BF16) FN<DT_BF16, DT_BF16>(__VA_ARGS__);                      \
        else if (at_ == DT_F32) FN<DT_Q4B32, DT_F32>(__VA_ARGS__);                       \
        else FN<DT_Q4B32, DT_BF16>(__VA_ARGS__);                                         \
    } while (0)

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D bf16 tensor [rows][cols] (cols contiguous), box = 64 columns x box_rows rows, 128-byte swizzle,
// out-of-range elements read as zero
bool make_map(const s2moe_ctx *ctx, CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    if (!ctx->encode_tiled || !base || rows == 0) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return ((EncodeTiledFn)ctx->encode_tiled)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims,
                                              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D tensor of `elem_bytes`-wide elements [rows][cols], box = box_cols x 128 rows (packed int4
// weights as bytes, their scales as 16-bit words); out-of-range elements read as zero.  Byte boxes
// of 32, 64 or 128 bytes are swizzled over their own width, so that threads which each read one
// 16-byte chunk of consecutive rows do not meet in the same shared-memory banks.
bool make_map_plain(const s2moe_ctx *ctx, CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols,
                    uint32_t box_cols, int elem_bytes)
{
    if (!ctx->encode_tiled || !base || rows == 0) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * (uint64_t)elem_bytes};
    const cuuint32_t box[2] = {box_cols, 128};
    const cuuint32_t estr[2] = {1, 1};
    return ((EncodeTiledFn)ctx->encode_tiled)(out, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_UINT16,
                                              2, const_cast<void *>(base), dims, strides, box, estr,
                                              CU_TENSOR_MAP_INTERLEAVE_NONE,
                                              elem_bytes != 1   ? CU_TENSOR_MAP_SWIZZLE_NONE
                                              : box_cols == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                              : box_cols == 64  ? CU_TENSOR_MAP_SWIZZLE_64B
                                                                : CU_TENSOR_MAP_SWIZZLE_32B,
                                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D bf16 tensor {cols, rows, 2}: the hi array and, `plane_bytes` further, the lo array of the
// activations; box = 64 columns x 8 rows x both planes
bool make_map_hilo(const s2moe_ctx *ctx, CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols,
                   uint64_t plane_bytes)
{
    if (!ctx->encode_tiled || !base || rows == 0) return false;
    const cuuint64_t dims[3] = {cols, rows, 2};
    const cuuint64_t strides[2] = {cols * 2, plane_bytes};
    const cuuint32_t box[3] = {64, 8, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return ((EncodeTiledFn)ctx->encode_tiled)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims,
                                              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 weights as {64 columns, rows, k-tiles of 64 columns}, box = 64 x 128 x 2: two k-tiles of a
// 128-row block in one copy, each a 16 KiB tile with the 128-byte swizzle
bool make_map_w2(const s2moe_ctx *ctx, CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols)
{
    if (!ctx->encode_tiled || !base || rows == 0 || cols % 64) return false;
    const cuuint64_t dims[3] = {64, rows, cols / 64};
    const cuuint64_t strides[2] = {cols * 2, 128};
    const cuuint32_t box[3] = {64, 128, 2};
    const cuuint32_t estr[3] = {1, 1, 1};
    return ((EncodeTiledFn)ctx->encode_tiled)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims,
                                              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// int4 path: the hidden states as {64 columns, rows, k-tiles of 64 columns}, box = 64 x box_rows x kg:
// the token tiles of kg consecutive k-tiles in one copy, each tile box_rows x 128 bytes
bool make_map_ktiles(const s2moe_ctx *ctx, CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols,
                     uint32_t box_rows, uint32_t kg)
{
    if (!ctx->encode_tiled || !base || rows == 0 || cols % 64) return false;
    const cuuint64_t dims[3] = {64, rows, cols / 64};
    const cuuint64_t strides[2] = {cols * 2, 128};
    const cuuint32_t box[3] = {64, box_rows, kg};
    const cuuint32_t estr[3] = {1, 1, 1};
    return ((EncodeTiledFn)ctx->encode_tiled)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims,
                                              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// int4 path: the activations as {64 columns, rows, k-tiles, hi / lo}, box = 64 x 8 x kg x 2: per copy
// the hi rows of 8 slots for kg k-tiles and, behind them, their lo rows
bool make_map_hilo_ktiles(const s2moe_ctx *ctx, CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols,
                          uint64_t plane_bytes, uint32_t kg)
{
    if (!ctx->encode_tiled || !base || rows == 0 || cols % 64) return false;
    const cuuint64_t dims[4] = {64, rows, cols / 64, 2};
    const cuuint64_t strides[3] = {cols * 2, 128, plane_bytes};
    const cuuint32_t box[4] = {64, 8, kg, 2};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return ((EncodeTiledFn)ctx->encode_tiled)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims,
                                              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The plan a batch of B tokens runs with: the streaming kernel when it is allowed and its
// shared-memory layout fits, else the CUDA-core kernels; 0 when plan 2 was demanded and does not fit.
int plan_for(const s2moe_ctx *ctx, int B, StPlan *out)
{
    const Shape &s0 = ctx->shape;
    const int want = ctx->cfg.kernel_plan;
    if (want == 1) return 1;
    if (want == 4) {
        // the whole layer in one launch, on demand only: measured slower than routing kernel + expert
        // kernel on every workload here (the gating runs two to three times longer inside the busy
        // CTAs than on a block of its own, and delays the first hand-over between the projections).
        // An offloaded context meets the host between routing and the experts: two launches.
        if (ctx->offload || ctx->tc_maps.empty()) return 0;
        const fused::TcPlan tp = fused::tc_make_plan(s0, B, ctx->n_sm, B * s0.k + s0.n_sh * B);
        return tp.feasible ? 4 : 0;
    }
    if (want == 0 || want == 3) {
        const TcPlan tp = tc_make_plan(s0, B, ctx->n_sm, B * s0.k + s0.n_sh * B, B >= ctx->bf16_kg2_from ? 2 : 1);
        if (tp.feasible && !ctx->tc_maps.empty()) return 3;
        if (want == 3) return 0;
    }
    const StPlan pl = st_make_plan(s0, B, ctx->n_sm, B * s0.k + s0.n_sh * B);
    if (out) *out = pl;
    if (pl.feasible) return 2;
    return want == 2 ? 0 : 1;
}

// Expert offloading, between the routing kernel and the FFN kernel of a layer: read the list of
// active experts back, let the layer's cache name a slot for each, copy the missing ones from
// host memory into their slots and hand the expert-to-slot table to the FFN kernel.  Host and
// stream meet here (the host has to see the routing result), so an offloaded layer is not
// captured into a graph.
int fetch_experts(s2moe_ctx *ctx, int layer, cudaStream_t st)
{
    const Shape &sh = ctx->shape;
    const int G = sh.E + sh.n_sh;
    CU(ctx, cudaMemcpyAsync(ctx->h_route, ctx->ws.header, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CU(ctx, cudaMemcpyAsync(ctx->h_route + 8, ctx->ws.active, (size_t)G * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CU(ctx, cudaStreamSynchronize(st));
    const int U = ctx->h_route[2];
    if (U < 0 || U > sh.E) return S2MOE_ECUDA;
    ExpertCache &cache = ctx->caches[(size_t)layer];
    std::vector<int32_t> slots((size_t)U), missed((size_t)U);
    if (!cache.access(ctx->h_route + 8, U, slots.data(), missed.data())) return S2MOE_ERANGE;
    const LayerPtrs &hw = ctx->host_w[(size_t)layer], &dw = ctx->layers[(size_t)layer];
    const void *src[6] = {hw.w_gate, hw.w_up, hw.w_down, hw.s_gate, hw.s_up, hw.s_down};
    const void *dst[6] = {dw.w_gate, dw.w_up, dw.w_down, dw.s_gate, dw.s_up, dw.s_down};
    // the cache already counts the missing experts as resident: if a copy cannot be issued, every
    // expert whose copies are not all on the stream is taken out again, so that a later call
    // fetches it instead of reading a slot that holds another expert's weights
    for (int i = 0; i < U; ++i) {
        if (!missed[(size_t)i]) continue;
        const size_t e = (size_t)ctx->h_route[8 + i], sl = (size_t)slots[(size_t)i];
        for (int m = 0; m < 6; ++m) {
            const size_t nb = ctx->mat_bytes[m];
            if (!nb) continue;
            const cudaError_t ce = cudaMemcpyAsync((uint8_t *)const_cast<void *>(dst[m]) + nb * sl,
                                                   (const uint8_t *)src[m] + nb * e, nb, cudaMemcpyHostToDevice, st);
            if (ce != cudaSuccess) {
                for (int j = i; j < U; ++j)
                    if (missed[(size_t)j]) cache.evict(ctx->h_route[8 + j]);
                return cuda_fail(ctx, ce);
            }
            ctx->fetched_bytes += (int64_t)nb;
        }
    }
    for (int e = 0; e < sh.E; ++e) ctx->h_slot_of[e] = cache.slot_of[(size_t)e] < 0 ? 0 : cache.slot_of[(size_t)e];
    CU(ctx, cudaMemcpyAsync(ctx->d_slot_of, ctx->h_slot_of, (size_t)sh.E * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    // h_slot_of is reused by the next call: the copy must have left the host buffer
    CU(ctx, cudaStreamSynchronize(st));
    return S2MOE_OK;
}

int verify_one(s2moe_ctx *ctx, int layer, int B, const void *hidden, const float *conf, float *out,
               int32_t *sel_idx, float *sel_w, int32_t *n_unique, cudaStream_t st)
{
    Shape sh = ctx->shape;
    const LayerPtrs &lp = ctx->layers[layer];
    StPlan pl{};
    const int plan = plan_for(ctx, B, &pl);
    if (plan == 0) return S2MOE_EINVAL;
    sh.plan = plan;
    sh.op_cap = pl.op_cap;
    // tensor-core plan with bf16 weights: the expert kernel starts while the gating still runs, on the
    // experts the routing kernel announces before it (not with offloaded experts: their weights are
    // fetched between the two kernels)
    const bool want_early = plan == 3 && ctx->early_start && ctx->use_pdl && !ctx->offload && sh.weight_dtype == DT_BF16;
    TcPlan tp3 = tc_make_plan(sh, B, ctx->n_sm, B * sh.k + sh.n_sh * B, B >= ctx->bf16_kg2_from ? 2 : 1, want_early);
    if (sh.weight_dtype == DT_BF16 && ctx->wave_split[0] > 0) { tp3.split[0] = ctx->wave_split[0]; tp3.split[1] = ctx->wave_split[1]; }
    // what the FFN kernels accumulate into is cleared by the routing kernel's blocks
    ZeroList zl{};
    zl.ptr[0] = out;
    zl.n16[0] = (size_t)B * sh.d * sizeof(float) / 16;
    if (plan == 3 || plan == 4) {
        const size_t used = (size_t)B * sh.k * sh.f + (size_t)sh.n_sh * B * sh.f_sh;
        zl.ptr[1] = ctx->pre;
        zl.n16[1] = used * 2 * sizeof(float) / 16;
        zl.ptr[2] = ctx->ws.sync + (kTcReady - 8);      // the hand-over counters of the two waves
        zl.n16[2] = 8 * sizeof(int32_t) / 16;
        if (sh.weight_dtype == DT_Q4B32) {
            zl.perm_src = (const uint4 *)hidden;
            zl.perm_dst = (uint4 *)ctx->hperm;
            zl.perm_n16 = (size_t)B * sh.d * 2 / 16;
        }
    }
    if (plan == 3 && tp3.early) {
        // a token's first expert by original logit stays selected for alpha < 1 (see gating_block);
        // otherwise only the shared experts start early
        const bool bias_on = sh.alpha > 0.0 && sh.cap < sh.E && sh.k < sh.E;
        zl.early = (!bias_on || sh.alpha <= 0.999999) ? 2 : 1;
    }
    if (plan != 4) launch_route(ctx, sh, lp, B, hidden, conf, sel_idx, sel_w, n_unique, zl, st);
    if (ctx->offload) {
        const int rc = fetch_experts(ctx, layer, st);
        if (rc != S2MOE_OK) return rc;
    }
    if (plan == 3 || plan == 4) {

        const fused::TcPlan tp4 = plan == 4 ? fused::tc_make_plan(sh, B, ctx->n_sm, B * sh.k + sh.n_sh * B) : fused::TcPlan{};
        const bool q4 = plan == 4 ? tp4.q4 != 0 : tp3.q4 != 0;
        const int tokb = plan == 4 ? tp4.tokb : tp3.tokb, kg = plan == 4 ? tp4.kg : tp3.kg;
        TcMaps maps = ctx->tc_maps[layer];
        const size_t n_routed = (size_t)B * sh.k;
        const uint64_t plane = (uint64_t)((const uint8_t *)ctx->act_lo - (const uint8_t *)ctx->act_hi);
        bool ok;
        if (q4) {
            ok = make_map_ktiles(ctx, &maps.m[6], ctx->hperm, (uint64_t)B, (uint64_t)sh.d, (uint32_t)tokb / 128, (uint32_t)kg) &&
                 make_map_hilo_ktiles(ctx, &maps.m[7], ctx->act_hi, n_routed, (uint64_t)sh.f, plane, (uint32_t)kg);
            if (ok && sh.n_sh)
                ok = make_map_hilo_ktiles(ctx, &maps.m[8], ctx->act_hi + n_routed * sh.f, (uint64_t)sh.n_sh * B,
                                          (uint64_t)sh.f_sh, plane, (uint32_t)kg);
        } else if (plan == 3 && tp3.kg == 2) {
            // two k-tiles per stage: the token tiles of both in one copy (see make_map_ktiles)
            // (resident hidden-state tiles are loaded once, k-tile by k-tile, through the plain 2-D map)
            ok = (tp3.x_bytes ? make_map(ctx, &maps.m[6], hidden, (uint64_t)B, (uint64_t)sh.d, (uint32_t)tp3.rows1)
                              : make_map_ktiles(ctx, &maps.m[6], hidden, (uint64_t)B, (uint64_t)sh.d, (uint32_t)tp3.tokb / 128, 2)) &&
                 make_map_hilo_ktiles(ctx, &maps.m[7], ctx->act_hi, n_routed, (uint64_t)sh.f, plane, 2);
            if (ok && sh.n_sh)
                ok = make_map_hilo_ktiles(ctx, &maps.m[8], ctx->act_hi + n_routed * sh.f, (uint64_t)sh.n_sh * B,
                                          (uint64_t)sh.f_sh, plane, 2);
        } else {
            ok = make_map(ctx, &maps.m[6], hidden, (uint64_t)B, (uint64_t)sh.d, plan == 3 ? (uint32_t)tp3.rows1 : 16u) &&
                 make_map_hilo(ctx, &maps.m[7], ctx->act_hi, n_routed, (uint64_t)sh.f, plane);
            if (ok && sh.n_sh)
                ok = make_map_hilo(ctx, &maps.m[8], ctx->act_hi + n_routed * sh.f, (uint64_t)sh.n_sh * B, (uint64_t)sh.f_sh, plane);
        }
        if (!ok) return S2MOE_ECUDA;
        if (plan == 3) {
            TcArgs a;
            a.sh = sh; a.ws = ctx->ws; a.plan = tp3; a.y = out; a.pre = ctx->pre;
            a.act_hi = ctx->act_hi; a.act_lo = ctx->act_lo; a.B = B; a.early = tp3.early;
            LaunchScope scope(ctx, KC_TC, st);
            cudaLaunchConfig_t lc = pdl_config(ctx, tp3.n_cta, q4 ? kTcQ4Threads : kTcThreads, tp3.smem_bytes, st, tp3.early != 0);
            if (q4) cudaLaunchKernelEx(&lc, ffn_tc_kernel<true>, maps, a);
            else cudaLaunchKernelEx(&lc, ffn_tc_kernel<false>, maps, a);
        } else {
            fused::TcArgs a;
            a.sh = sh; a.ws = ctx->ws; a.plan = tp4; a.y = out; a.pre = ctx->pre;
            a.act_hi = ctx->act_hi; a.act_lo = ctx->act_lo; a.B = B;
            a.sh.plan = 3;
            a.rt = fused::TcRoute{};
            a.rt.hidden = hidden; a.rt.router = lp.router; a.rt.sh_scale = lp.sh_scale; a.rt.conf = conf;
            a.rt.sel_idx = sel_idx; a.rt.sel_w = sel_w; a.rt.n_unique = n_unique;
            a.rt.lpart = ctx->lpart;
            a.rt.gbar = reinterpret_cast<unsigned long long *>(ctx->ws.ticket + 4);
            a.rt.zl = zl;
            // the expert of a token's largest logit stays in its top-k under any bias of alpha <= 1
            const bool bias_on = sh.alpha > 0.0 && sh.cap < sh.E && sh.k < sh.E;
            a.rt.early = (!bias_on || sh.alpha <= 1.0) ? 1 : 0;
            LaunchScope scope(ctx, KC_LAYER, st);
            cudaLaunchConfig_t lc = pdl_config(ctx, tp4.n_cta, q4 ? kTcQ4Threads : kTcThreads, tp4.smem_bytes, st);
            if (q4) cudaLaunchKernelEx(&lc, fused::layer_tc_kernel<true>, maps, a);
            else cudaLaunchKernelEx(&lc, fused::layer_tc_kernel<false>, maps, a);
        }
    } else if (plan == 2) {
        StreamArgs a;
        a.sh = sh; a.lp = lp; a.ws = ctx->ws; a.plan = pl; a.hidden = hidden; a.y = out;
        a.act_hi = ctx->act_hi; a.act_lo = ctx->act_lo; a.B = B;
        a.act_elems = ctx->act_elems;
        LaunchScope scope(ctx, KC_STREAM, st);
        ffn_stream_kernel<<<pl.n_cta, kStThreads, pl.smem_bytes, st>>>(a);
    } else {
        DISPATCH_WT_ACT(ctx, launch_simple, ctx, lp, hidden, out, st);
    }
    ctx->last_B = B;
    CU(ctx, cudaGetLastError());
    return S2MOE_OK;
}

int check_call(s2moe_ctx *ctx, int32_t n_tokens, const void *hidden, float *out, int32_t *sel_idx, float *sel_w,
               int32_t *n_unique)
{
    if (!ctx) return S2MOE_EINVAL;
    if (n_tokens < 0 || n_tokens > ctx->cfg.max_tokens) return S2MOE_ERANGE;
    if (n_tokens == 0) return S2MOE_OK;
    if (!hidden || !out || !sel_idx || !sel_w || !n_unique) return S2MOE_EINVAL;
    if (!aligned16(hidden) || !aligned16(out)) return S2MOE_EINVAL;
    return S2MOE_OK;
}

}  // namespace

extern "C" {

namespace {
int create_impl(const s2moe_config *config, const s2moe_layer_weights *layers, int n_w_experts, s2moe_ctx **out);
}

int s2moe_create(const s2moe_config *config, const s2moe_layer_weights *layers, s2moe_ctx **out)
{
    if (out) *out = nullptr;
    if (!config || !layers || !out) return S2MOE_EINVAL;
    return create_impl(config, layers, config->n_experts, out);
}

namespace {
// n_w_experts: how many experts the routed-expert weight tensors of `layers` hold (all of them,
// or the slots of the device pool of an offloaded context)
int create_impl(const s2moe_config *config, const s2moe_layer_weights *layers, int n_w_experts, s2moe_ctx **out)
{
    if (out) *out = nullptr;
    if (!config || !layers || !out) return S2MOE_EINVAL;
    int rc = validate_config(config);
    if (rc != S2MOE_OK) return rc;
    for (int l = 0; l < config->n_layers; ++l) {
        rc = validate_layer(config, &layers[l]);
        if (rc != S2MOE_OK) return rc;
    }
    s2moe_ctx *ctx = new (std::nothrow) s2moe_ctx();
    if (!ctx) return S2MOE_ENOMEM;
    ctx->cfg = *config;
    ctx->n_w_experts = n_w_experts;
    Shape &sh = ctx->shape;
    sh.d = config->d_model; sh.f = config->d_ff; sh.E = config->n_experts; sh.k = config->top_k;
    sh.n_sh = config->n_shared; sh.f_sh = config->n_shared ? config->d_ff_shared : 0;
    sh.act_dtype = config->act_dtype; sh.router_dtype = config->router_dtype;
    sh.weight_dtype = config->weight_dtype;
    sh.renorm = config->renorm; sh.cap = config->cap; sh.weight_mode = config->weight_mode;
    sh.alpha = (double)config->alpha;
    ctx->layers.resize(config->n_layers);
    static_assert(sizeof(LayerPtrs) == sizeof(s2moe_layer_weights), "layout");
    std::memcpy(ctx->layers.data(), layers, sizeof(LayerPtrs) * (size_t)config->n_layers);
    ctx->plan = config->kernel_plan;
    sh.plan = 1;
    sh.op_cap = 0;

    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e != cudaSuccess) { delete ctx; return S2MOE_ECUDA; }

    const int T = config->max_tokens, E = sh.E, G = E + sh.n_sh, L = config->n_layers;
    const size_t n_slots = (size_t)T * sh.k + (size_t)sh.n_sh * T;
    const size_t act_floats = (size_t)T * sh.k * sh.f + (size_t)sh.n_sh * T * sh.f_sh;
    const size_t ab = sh.act_dtype == DT_F32 ? 4 : 2;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t o_logits = take(sizeof(double) * T * E), o_gl = take(sizeof(double) * T);
    const size_t o_ticket = take(256), o_status = take(256), o_header = take(256);
    const size_t o_counts = take(4 * (size_t)G), o_offsets = take(4 * (size_t)(G + 1));
    const size_t o_stok = take(4 * n_slots), o_sw = take(4 * n_slots), o_active = take(4 * (size_t)G);
    const size_t o_act = take(4 * act_floats), o_sync = take(4 * (size_t)(kTcReady + kStMaxGroups + 64));
    const size_t o_pre = take(8 * act_floats);
    const size_t o_ahi = take(2 * act_floats), o_alo = take(2 * act_floats);
    const size_t o_up1 = take(4 * (size_t)(G + 2)), o_up2 = take(4 * (size_t)(G + 2));
    const size_t o_tm = take(8 * (size_t)G);
    const size_t o_gtab = take(32 * (size_t)(G + 1));
    const size_t o_early = take(4 * (size_t)(kMaxTokens + 4));
    const size_t o_hperm = take(sh.weight_dtype == DT_Q4B32 ? 2 * (size_t)T * sh.d : 0);
    const size_t o_lpart = take(sizeof(double) * 8 * (size_t)T * (E + 1));
    const size_t o_sth = take(ab * (size_t)L * T * sh.d), o_stc = take(4 * (size_t)L * T);
    const size_t o_sto = take(4 * (size_t)L * T * sh.d), o_sts = take(4 * (size_t)L * T * sh.k);
    const size_t o_stw = take(4 * (size_t)L * T * sh.k), o_stn = take(4 * (size_t)L);
    ctx->slab_bytes = off;
    ctx->act_elems = act_floats;
    e = cudaMalloc(&ctx->slab, ctx->slab_bytes);
    if (e != cudaSuccess) { delete ctx; return e == cudaErrorMemoryAllocation ? S2MOE_ENOMEM : S2MOE_ECUDA; }
    e = cudaMemset(ctx->slab, 0, ctx->slab_bytes);
    if (e == cudaSuccess) DISPATCH_WT_ACT(ctx, e = prepare_simple);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->n_sm, cudaDevAttrMultiProcessorCount, ctx->device);
    {
        const char *no_pdl = std::getenv("S2MOE_NO_PDL");
        ctx->use_pdl = !(no_pdl && no_pdl[0] == '1');
        const char *kgv = std::getenv("S2MOE_BF16_KG2_FROM");
        if (kgv && std::atoi(kgv) > 0) ctx->bf16_kg2_from = std::atoi(kgv);
        const char *tf = std::getenv("S2MOE_ROUTE_TASKS_FROM");
        if (tf && tf[0]) ctx->route_task_from = std::atoi(tf);
        const char *pg = std::getenv("S2MOE_PDL_IN_GRAPH");
        ctx->pdl_in_graph = pg && pg[0] == '1';
        const char *wv = std::getenv("S2MOE_WAVES");
        if (wv && wv[0]) {
            int a = 0, b = 16;
            if (std::sscanf(wv, "%d,%d", &a, &b) >= 1 && a > 0 && a <= 16 && b >= a && b <= 16) { ctx->wave_split[0] = a; ctx->wave_split[1] = b; }
        }
        const char *ne = std::getenv("S2MOE_NO_EARLY");
        ctx->early_start = !(ne && ne[0] == '1');
    }
    if (e == cudaSuccess && ctx->plan != 1)
        e = cudaFuncSetAttribute(ffn_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStMaxSmem);
    if (e == cudaSuccess) e = prepare_route();
    if (e != cudaSuccess) { cudaFree(ctx->slab); delete ctx; return S2MOE_ECUDA; }
    uint8_t *base = (uint8_t *)ctx->slab;
    Workspace &ws = ctx->ws;
    ws.logits = (double *)(base + o_logits); ws.gate_logit = (double *)(base + o_gl);
    ws.ticket = (unsigned int *)(base + o_ticket); ws.status = (int32_t *)(base + o_status);
    ws.header = (int32_t *)(base + o_header); ws.counts = (int32_t *)(base + o_counts);
    ws.offsets = (int32_t *)(base + o_offsets); ws.slot_token = (int32_t *)(base + o_stok);
    ws.slot_w = (float *)(base + o_sw); ws.active = (int32_t *)(base + o_active);
    ws.act = (float *)(base + o_act); ws.sync = (int32_t *)(base + o_sync);
    ws.upfx1 = (int32_t *)(base + o_up1); ws.upfx2 = (int32_t *)(base + o_up2);
    ws.tokmask = (unsigned long long *)(base + o_tm);
    ws.gtab = (uint4 *)(base + o_gtab);
    ws.early = (int32_t *)(base + o_early);
    ctx->hperm = base + o_hperm;
    ctx->lpart = (double *)(base + o_lpart);
    ctx->pre = (float *)(base + o_pre);
    // plan 3: tensor maps of the weights (one set per layer); without the driver entry point or
    // for other formats the plan is simply not offered
    if (ctx->plan != 1 && ctx->plan != 2 && (sh.weight_dtype == DT_BF16 || sh.weight_dtype == DT_Q4B32) &&
        sh.act_dtype == DT_BF16) {
        cudaDriverEntryPointQueryResult qres;
        void *fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess && fn) {
            ctx->encode_tiled = fn;
            ctx->tc_maps.resize(config->n_layers);
            const bool q4 = sh.weight_dtype == DT_Q4B32;
            bool ok = cudaFuncSetAttribute(ffn_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcMaxSmem) == cudaSuccess &&
                      cudaFuncSetAttribute(ffn_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcMaxSmem) == cudaSuccess &&
                      cudaFuncSetAttribute(fused::layer_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcMaxSmem) == cudaSuccess &&
                      cudaFuncSetAttribute(fused::layer_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcMaxSmem) == cudaSuccess;
            // the int4 variant needs contraction lengths that are multiples of 256 (see tc_make_plan)
            if (q4 && (sh.d % 256 || sh.f % 256 || (sh.n_sh && sh.f_sh % 256))) ok = false;
            for (int l = 0; l < config->n_layers && ok; ++l) {
                const LayerPtrs &lp = ctx->layers[l];
                TcMaps &m = ctx->tc_maps[l];
                std::memset(&m, 0, sizeof(m));
                if (q4) {
                    const uint64_t Ef = (uint64_t)n_w_experts * sh.f, Ed = (uint64_t)n_w_experts * sh.d;
                    ok = make_map_plain(ctx, &m.m[0], lp.w_gate, Ef, (uint64_t)sh.d / 2, 32, 1) &&
                         make_map_plain(ctx, &m.m[1], lp.w_up, Ef, (uint64_t)sh.d / 2, 32, 1) &&
                         make_map_plain(ctx, &m.m[2], lp.w_down, Ed, (uint64_t)sh.f / 2, 32, 1) &&
                         make_map_plain(ctx, &m.m[9], lp.s_gate, Ef, (uint64_t)sh.d / 32, 8, 2) &&
                         make_map_plain(ctx, &m.m[10], lp.s_up, Ef, (uint64_t)sh.d / 32, 8, 2) &&
                         make_map_plain(ctx, &m.m[11], lp.s_down, Ed, (uint64_t)sh.f / 32, 8, 2);
                    // the packed matrices again with boxes of two and of four k-tiles
                    for (int j = 1; j <= 2 && ok; ++j) {
                        const int base = 15 + 6 * (j - 1);
                        const uint32_t bc = 32u << j;
                        ok = make_map_plain(ctx, &m.m[base + 0], lp.w_gate, Ef, (uint64_t)sh.d / 2, bc, 1) &&
                             make_map_plain(ctx, &m.m[base + 1], lp.w_up, Ef, (uint64_t)sh.d / 2, bc, 1) &&
                             make_map_plain(ctx, &m.m[base + 2], lp.w_down, Ed, (uint64_t)sh.f / 2, bc, 1);
                        if (ok && sh.n_sh) {
                            const uint64_t Sf = (uint64_t)sh.n_sh * sh.f_sh, Sd = (uint64_t)sh.n_sh * sh.d;
                            ok = make_map_plain(ctx, &m.m[base + 3], lp.sh_gate, Sf, (uint64_t)sh.d / 2, bc, 1) &&
                                 make_map_plain(ctx, &m.m[base + 4], lp.sh_up, Sf, (uint64_t)sh.d / 2, bc, 1) &&
                                 make_map_plain(ctx, &m.m[base + 5], lp.sh_down, Sd, (uint64_t)sh.f_sh / 2, bc, 1);
                        }
                    }
                    if (ok && sh.n_sh) {
                        const uint64_t Sf = (uint64_t)sh.n_sh * sh.f_sh, Sd = (uint64_t)sh.n_sh * sh.d;
                        ok = make_map_plain(ctx, &m.m[3], lp.sh_gate, Sf, (uint64_t)sh.d / 2, 32, 1) &&
                             make_map_plain(ctx, &m.m[4], lp.sh_up, Sf, (uint64_t)sh.d / 2, 32, 1) &&
                             make_map_plain(ctx, &m.m[5], lp.sh_down, Sd, (uint64_t)sh.f_sh / 2, 32, 1) &&
                             make_map_plain(ctx, &m.m[12], lp.sh_s_gate, Sf, (uint64_t)sh.d / 32, 8, 2) &&
                             make_map_plain(ctx, &m.m[13], lp.sh_s_up, Sf, (uint64_t)sh.d / 32, 8, 2) &&
                             make_map_plain(ctx, &m.m[14], lp.sh_s_down, Sd, (uint64_t)sh.f_sh / 32, 8, 2);
                    }
                    continue;
                }
                ok = make_map(ctx, &m.m[0], lp.w_gate, (uint64_t)n_w_experts * sh.f, (uint64_t)sh.d, 128) &&
                     make_map(ctx, &m.m[1], lp.w_up, (uint64_t)n_w_experts * sh.f, (uint64_t)sh.d, 128) &&
                     make_map(ctx, &m.m[2], lp.w_down, (uint64_t)n_w_experts * sh.d, (uint64_t)sh.f, 128);
                if (ok && sh.n_sh)
                    ok = make_map(ctx, &m.m[3], lp.sh_gate, (uint64_t)sh.n_sh * sh.f_sh, (uint64_t)sh.d, 128) &&
                         make_map(ctx, &m.m[4], lp.sh_up, (uint64_t)sh.n_sh * sh.f_sh, (uint64_t)sh.d, 128) &&
                         make_map(ctx, &m.m[5], lp.sh_down, (uint64_t)sh.n_sh * sh.d, (uint64_t)sh.f_sh, 128);
                // the same matrices with two k-tiles per copy (maps 9..14), where every contraction
                // length is a multiple of 64
                if (ok && sh.d % 64 == 0 && sh.f % 64 == 0 && (sh.n_sh == 0 || sh.f_sh % 64 == 0)) {
                    ok = make_map_w2(ctx, &m.m[9], lp.w_gate, (uint64_t)n_w_experts * sh.f, (uint64_t)sh.d) &&
                         make_map_w2(ctx, &m.m[10], lp.w_up, (uint64_t)n_w_experts * sh.f, (uint64_t)sh.d) &&
                         make_map_w2(ctx, &m.m[11], lp.w_down, (uint64_t)n_w_experts * sh.d, (uint64_t)sh.f);
                    if (ok && sh.n_sh)
                        ok = make_map_w2(ctx, &m.m[12], lp.sh_gate, (uint64_t)sh.n_sh * sh.f_sh, (uint64_t)sh.d) &&
                             make_map_w2(ctx, &m.m[13], lp.sh_up, (uint64_t)sh.n_sh * sh.f_sh, (uint64_t)sh.d) &&
                             make_map_w2(ctx, &m.m[14], lp.sh_down, (uint64_t)sh.n_sh * sh.d, (uint64_t)sh.f_sh);
                }
            }
            if (!ok) ctx->tc_maps.clear();
        }
    }
    ctx->act_hi = (__nv_bfloat16 *)(base + o_ahi); ctx->act_lo = (__nv_bfloat16 *)(base + o_alo);
    ctx->st_hidden = base + o_sth; ctx->st_conf = (float *)(base + o_stc);
    ctx->st_out = (float *)(base + o_sto); ctx->st_sel = (int32_t *)(base + o_sts);
    ctx->st_selw = (float *)(base + o_stw); ctx->st_nu = (int32_t *)(base + o_stn);
    *out = ctx;
    return S2MOE_OK;
}
}  // namespace

int s2moe_create_offloaded(const s2moe_config *config, const s2moe_layer_weights *layers, const s2moe_residency *res,
                           s2moe_ctx **out)
{
    if (out) *out = nullptr;
    if (!config || !layers || !res || !out) return S2MOE_EINVAL;
    int rc = validate_config(config);
    if (rc != S2MOE_OK) return rc;
    const int E = config->n_experts, L = config->n_layers;
    if (res->n_slots < 1 || res->n_slots > E || res->n_pinned < 0 || res->n_pinned > res->n_slots) return S2MOE_EINVAL;
    if (res->n_pinned > 0 && !res->pinned) return S2MOE_EINVAL;
    // the expert-to-slot indirection lives in the tcgen05 kernel
    if (config->kernel_plan != 0 && config->kernel_plan != 3) return S2MOE_EINVAL;
    if (config->act_dtype != S2MOE_BF16 || (config->weight_dtype != S2MOE_BF16 && config->weight_dtype != S2MOE_Q4B32))
        return S2MOE_EINVAL;
    for (int l = 0; l < L; ++l) {
        rc = validate_layer(config, &layers[l]);     // non-null and 16-byte aligned holds for host pointers too
        if (rc != S2MOE_OK) return rc;
    }
    const bool q4 = config->weight_dtype == S2MOE_Q4B32;
    const size_t d = (size_t)config->d_model, f = (size_t)config->d_ff;
    size_t mb[6] = {0, 0, 0, 0, 0, 0};
    mb[0] = mb[1] = mb[2] = q4 ? f * d / 2 : f * d * 2;
    if (q4) mb[3] = mb[4] = mb[5] = f * (d / 32) * 2;
    size_t per_layer = 0;
    for (int i = 0; i < 6; ++i) per_layer += align_up(mb[i] * (size_t)res->n_slots, 256);
    void *pool = nullptr;
    cudaError_t e = cudaMalloc(&pool, per_layer * (size_t)L);
    if (e != cudaSuccess) return e == cudaErrorMemoryAllocation ? S2MOE_ENOMEM : S2MOE_ECUDA;
    std::vector<s2moe_layer_weights> dev((size_t)L);
    for (int l = 0; l < L; ++l) {
        dev[(size_t)l] = layers[l];
        uint8_t *p = (uint8_t *)pool + per_layer * (size_t)l;
        const void **dst[6] = {&dev[(size_t)l].w_gate, &dev[(size_t)l].w_up, &dev[(size_t)l].w_down,
                               &dev[(size_t)l].s_gate, &dev[(size_t)l].s_up, &dev[(size_t)l].s_down};
        for (int i = 0; i < 6; ++i) {
            if (mb[i]) *dst[i] = p;
            p += align_up(mb[i] * (size_t)res->n_slots, 256);
        }
    }
    s2moe_config cfg3 = *config;
    cfg3.kernel_plan = 3;
    s2moe_ctx *ctx = nullptr;
    rc = create_impl(&cfg3, dev.data(), res->n_slots, &ctx);
    if (rc != S2MOE_OK) { cudaFree(pool); return rc; }
    ctx->pool = pool;
    ctx->offload = true;
    for (int i = 0; i < 6; ++i) ctx->mat_bytes[i] = mb[i];
    ctx->host_w.resize((size_t)L);
    std::memcpy(ctx->host_w.data(), layers, sizeof(LayerPtrs) * (size_t)L);
    // every batch size up to max_tokens must run on the tcgen05 kernel
    bool ok = !ctx->tc_maps.empty();
    for (int B = 1; B <= config->max_tokens && ok; ++B) ok = plan_for(ctx, B, nullptr) == 3;
    ctx->caches.resize((size_t)L);
    for (int l = 0; l < L && ok; ++l)
        ok = ctx->caches[(size_t)l].init(E, res->n_slots, res->n_pinned ? res->pinned + (size_t)l * res->n_pinned : nullptr,
                                         res->n_pinned);
    if (!ok) { s2moe_destroy(ctx); return S2MOE_EINVAL; }
    e = cudaMallocHost((void **)&ctx->h_route, sizeof(int32_t) * (size_t)(8 + E + config->n_shared));
    if (e == cudaSuccess) e = cudaMallocHost((void **)&ctx->h_slot_of, sizeof(int32_t) * (size_t)E);
    if (e == cudaSuccess) e = cudaMalloc((void **)&ctx->d_slot_of, sizeof(int32_t) * (size_t)E);
    // the pinned experts go to their slots now
    for (int l = 0; l < L && e == cudaSuccess; ++l) {
        const LayerPtrs &hw = ctx->host_w[(size_t)l], &dw = ctx->layers[(size_t)l];
        const void *src[6] = {hw.w_gate, hw.w_up, hw.w_down, hw.s_gate, hw.s_up, hw.s_down};
        const void *dstp[6] = {dw.w_gate, dw.w_up, dw.w_down, dw.s_gate, dw.s_up, dw.s_down};
        for (int i = 0; i < res->n_pinned && e == cudaSuccess; ++i) {
            const size_t ex = (size_t)res->pinned[(size_t)l * res->n_pinned + i];
            for (int m = 0; m < 6 && e == cudaSuccess; ++m)
                if (mb[m])
                    e = cudaMemcpy((uint8_t *)const_cast<void *>(dstp[m]) + mb[m] * (size_t)i,
                                   (const uint8_t *)src[m] + mb[m] * ex, mb[m], cudaMemcpyHostToDevice);
        }
    }
    if (e != cudaSuccess) { s2moe_destroy(ctx); return e == cudaErrorMemoryAllocation ? S2MOE_ENOMEM : S2MOE_ECUDA; }
    ctx->ws.slot_of = ctx->d_slot_of;
    *out = ctx;
    return S2MOE_OK;
}

int s2moe_residency_stats(const s2moe_ctx *ctx, int64_t *hits, int64_t *misses, int64_t *bytes_fetched)
{
    if (!ctx || !ctx->offload) return S2MOE_EINVAL;
    int64_t h = 0, m = 0;
    for (const ExpertCache &c : ctx->caches) { h += c.hits; m += c.misses; }
    if (hits) *hits = h;
    if (misses) *misses = m;
    if (bytes_fetched) *bytes_fetched = ctx->fetched_bytes;
    return S2MOE_OK;
}

int s2moe_residency_uses(const s2moe_ctx *ctx, int32_t layer, int64_t *uses_out)
{
    if (!ctx || !ctx->offload || !uses_out) return S2MOE_EINVAL;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return S2MOE_ERANGE;
    const ExpertCache &c = ctx->caches[(size_t)layer];
    for (int e = 0; e < c.n_experts; ++e) uses_out[e] = c.uses[(size_t)e];
    return S2MOE_OK;
}

int s2moe_cache_create(int32_t n_experts, int32_t n_slots, const int32_t *pinned, int32_t n_pinned, s2moe_cache **out)
{
    if (out) *out = nullptr;
    if (!out) return S2MOE_EINVAL;
    s2moe_cache *c = new (std::nothrow) s2moe_cache();
    if (!c) return S2MOE_ENOMEM;
    if (!c->c.init(n_experts, n_slots, pinned, n_pinned)) { delete c; return S2MOE_EINVAL; }
    *out = c;
    return S2MOE_OK;
}

int s2moe_cache_access(s2moe_cache *cache, const int32_t *experts, int32_t n, int32_t *slots_out, int32_t *missed_out)
{
    if (!cache || (n > 0 && (!experts || !slots_out || !missed_out))) return S2MOE_EINVAL;
    return cache->c.access(experts, n, slots_out, missed_out) ? S2MOE_OK : S2MOE_ERANGE;
}

int s2moe_cache_destroy(s2moe_cache *cache)
{
    delete cache;
    return S2MOE_OK;
}

int s2moe_verify_layer(s2moe_ctx *ctx, int32_t layer, int32_t n_tokens, const void *hidden, const float *conf,
                       float *out, int32_t *sel_idx, float *sel_w, int32_t *n_unique, void *cuda_stream)
{
    int rc = check_call(ctx, n_tokens, hidden, out, sel_idx, sel_w, n_unique);
    if (rc != S2MOE_OK) return rc;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return S2MOE_ERANGE;
    if (n_tokens == 0) return S2MOE_OK;
    return verify_one(ctx, layer, n_tokens, hidden, conf, out, sel_idx, sel_w, n_unique,
                      (cudaStream_t)cuda_stream);
}

int s2moe_verify_stack(s2moe_ctx *ctx, int32_t n_tokens, const void *hidden, const float *conf, float *out,
                       int32_t *sel_idx, float *sel_w, int32_t *n_unique, void *cuda_stream)
{
    int rc = check_call(ctx, n_tokens, hidden, out, sel_idx, sel_w, n_unique);
    if (rc != S2MOE_OK || n_tokens == 0) return rc;
    const Shape &sh = ctx->shape;
    const size_t ab = sh.act_dtype == DT_F32 ? 4 : 2, B = (size_t)n_tokens;
    for (int l = 0; l < ctx->cfg.n_layers; ++l) {
        rc = verify_one(ctx, l, n_tokens, (const uint8_t *)hidden + (size_t)l * B * sh.d * ab,
                        conf ? conf + (size_t)l * B : nullptr, out + (size_t)l * B * sh.d,
                        sel_idx + (size_t)l * B * sh.k, sel_w + (size_t)l * B * sh.k, n_unique + l,
                        (cudaStream_t)cuda_stream);
        if (rc != S2MOE_OK) return rc;
    }
    return S2MOE_OK;
}

int s2moe_verify_stack_host(s2moe_ctx *ctx, int32_t n_tokens, const void *hidden_host, const float *conf_host,
                            float *out_host, int32_t *sel_idx_host, float *sel_w_host, int32_t *n_unique_host,
                            void *cuda_stream)
{
    if (!ctx) return S2MOE_EINVAL;
    if (n_tokens < 0 || n_tokens > ctx->cfg.max_tokens) return S2MOE_ERANGE;
    if (n_tokens == 0) return S2MOE_OK;
    if (!hidden_host || !out_host || !sel_idx_host || !sel_w_host || !n_unique_host) return S2MOE_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const Shape &sh = ctx->shape;
    const size_t ab = sh.act_dtype == DT_F32 ? 4 : 2, L = (size_t)ctx->cfg.n_layers, B = (size_t)n_tokens;
    // The copies run beside the kernels.  In: the first layer's inputs go ahead on the caller's
    // stream, the other layers' follow on a stream of their own once the first layer is launched.
    // Out: the outputs of the layers up to the middle of the stack, and of those up to the last but
    // one, leave on a third stream while the later layers run; after the last kernel the last
    // layer's outputs and, in one copy into page-locked memory of the context, the indices, weights
    // and counts of all layers travel on two streams at once.
    if (!ctx->cs_in) CU(ctx, cudaStreamCreateWithFlags(&ctx->cs_in, cudaStreamNonBlocking));
    if (!ctx->cs_out) CU(ctx, cudaStreamCreateWithFlags(&ctx->cs_out, cudaStreamNonBlocking));
    for (cudaEvent_t &ev : ctx->ev_copy)
        if (!ev) CU(ctx, cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    // st_sel, st_selw and st_nu lie one after the other in the workspace, sized for max_tokens: this
    // call packs its indices, weights and counts at the front of that region
    const size_t region = (size_t)((const uint8_t *)(ctx->st_nu + L) - (const uint8_t *)ctx->st_sel);
    if (!ctx->h_small) CU(ctx, cudaHostAlloc((void **)&ctx->h_small, region, cudaHostAllocDefault));
    const size_t nsel = L * B * sh.k * 4, small_bytes = 2 * nsel + L * 4;
    uint8_t *const d_small = (uint8_t *)ctx->st_sel;
    int32_t *const d_sel = (int32_t *)d_small, *const d_nu = (int32_t *)(d_small + 2 * nsel);
    float *const d_selw = (float *)(d_small + nsel);
    const size_t hb = B * sh.d * ab;
    const int nl = (int)L;
    CU(ctx, cudaMemcpyAsync(ctx->st_hidden, hidden_host, hb, cudaMemcpyHostToDevice, st));
    if (conf_host) CU(ctx, cudaMemcpyAsync(ctx->st_conf, conf_host, L * B * 4, cudaMemcpyHostToDevice, st));
    auto copy_out = [&](int lo, int hi, cudaStream_t cs) -> int {      // outputs of layers lo .. hi - 1
        const size_t o = (size_t)lo * B * sh.d, n = (size_t)(hi - lo) * B * sh.d;
        CU(ctx, cudaMemcpyAsync(out_host + o, ctx->st_out + o, n * 4, cudaMemcpyDeviceToHost, cs));
        return S2MOE_OK;
    };
    const int cut1 = nl >= 4 ? nl / 2 : 0, cut2 = nl >= 2 ? nl - 1 : 0;   // layers copied early: [0, cut1), [cut1, cut2)
    int done = 0, rc = S2MOE_OK;
    for (int l = 0; l < nl && rc == S2MOE_OK; ++l) {
        if (l == 1) {
            CU(ctx, cudaMemcpyAsync((uint8_t *)ctx->st_hidden + hb, (const uint8_t *)hidden_host + hb, (L - 1) * hb,
                                    cudaMemcpyHostToDevice, ctx->cs_in));
            CU(ctx, cudaEventRecord(ctx->ev_copy[0], ctx->cs_in));
            CU(ctx, cudaStreamWaitEvent(st, ctx->ev_copy[0], 0));
        }
        rc = verify_one(ctx, l, n_tokens, (const uint8_t *)ctx->st_hidden + (size_t)l * hb,
                        conf_host ? ctx->st_conf + (size_t)l * B : nullptr, ctx->st_out + (size_t)l * B * sh.d,
                        d_sel + (size_t)l * B * sh.k, d_selw + (size_t)l * B * sh.k, d_nu + l, st);
        if (rc == S2MOE_OK && (l + 1 == cut1 || l + 1 == cut2) && l + 1 > done) {
            cudaEvent_t ev = ctx->ev_copy[l + 1 == cut1 ? 1 : 2];
            CU(ctx, cudaEventRecord(ev, st));
            CU(ctx, cudaStreamWaitEvent(ctx->cs_out, ev, 0));
            rc = copy_out(done, l + 1, ctx->cs_out);
            done = l + 1;
        }
    }
    if (rc == S2MOE_OK) {
        CU(ctx, cudaEventRecord(ctx->ev_copy[3], st));
        CU(ctx, cudaStreamWaitEvent(ctx->cs_out, ctx->ev_copy[3], 0));
        CU(ctx, cudaMemcpyAsync(ctx->h_small, d_small, small_bytes, cudaMemcpyDeviceToHost, ctx->cs_out));
        rc = copy_out(done, nl, st);
    }
    // all streams are drained whatever happened, so that no copy of this call outlives it
    const cudaError_t e1 = cudaStreamSynchronize(st), e2 = cudaStreamSynchronize(ctx->cs_out),
                      e3 = cudaStreamSynchronize(ctx->cs_in);
    if (rc != S2MOE_OK) return rc;
    CU(ctx, e1);
    CU(ctx, e2);
    CU(ctx, e3);
    const uint8_t *hs = ctx->h_small;
    memcpy(sel_idx_host, hs, nsel);
    memcpy(sel_w_host, hs + nsel, nsel);
    memcpy(n_unique_host, hs + 2 * nsel, L * 4);
    return S2MOE_OK;
}

int s2moe_destroy(s2moe_ctx *ctx)
{
    if (!ctx) return S2MOE_OK;
    cudaError_t e = cudaSuccess;
    if (ctx->slab) e = cudaFree(ctx->slab);
    if (ctx->pool) cudaFree(ctx->pool);
    if (ctx->d_slot_of) cudaFree(ctx->d_slot_of);
    if (ctx->h_route) cudaFreeHost(ctx->h_route);
    if (ctx->h_slot_of) cudaFreeHost(ctx->h_slot_of);
    for (cudaEvent_t ev : ctx->prof_ev) cudaEventDestroy(ev);
    for (cudaEvent_t ev : ctx->ev_copy) if (ev) cudaEventDestroy(ev);
    if (ctx->h_small) cudaFreeHost(ctx->h_small);
    if (ctx->cs_in) cudaStreamDestroy(ctx->cs_in);
    if (ctx->cs_out) cudaStreamDestroy(ctx->cs_out);
    delete ctx;
    return e == cudaSuccess ? S2MOE_OK : S2MOE_ECUDA;
}

const char *s2moe_strerror(int status)
{
    switch (status) {
        case S2MOE_OK: return "ok";
        case S2MOE_EINVAL: return "invalid argument (config, shape, null pointer or alignment)";
        case S2MOE_ERANGE: return "n_tokens or layer out of range, or more active experts than resident slots";
        case S2MOE_ENOMEM: return "out of device memory";
        case S2MOE_ECUDA: return "CUDA call failed";
        case S2MOE_ETIMEOUT: return "a bounded device-side wait gave up";
        default: return "unknown status";
    }
}

int s2moe_last_device_status(s2moe_ctx *ctx, int32_t *host_out)
{
    if (!ctx || !host_out) return S2MOE_EINVAL;
    CU(ctx, cudaDeviceSynchronize());
    CU(ctx, cudaMemcpy(host_out, ctx->ws.status, 4, cudaMemcpyDeviceToHost));
    if (*host_out != 0) {
        // the device is idle here: put the status word and the routing kernel's arrival words back,
        // so that the next call starts clean whatever the abandoned wait left behind
        CU(ctx, cudaMemset(ctx->ws.status, 0, 4));
        CU(ctx, cudaMemset(ctx->ws.ticket, 0, 16));
        return S2MOE_ETIMEOUT;
    }
    return S2MOE_OK;
}

int s2moe_last_cuda_error(const s2moe_ctx *ctx) { return ctx ? ctx->last_cuda : 0; }

int s2moe_kernel_plan(const s2moe_ctx *ctx, int32_t n_tokens)
{
    if (!ctx || n_tokens < 1 || n_tokens > ctx->cfg.max_tokens) return 0;
    return plan_for(ctx, n_tokens, nullptr);
}

int64_t s2moe_kernel_launches(const s2moe_ctx *ctx) { return ctx ? ctx->launches : 0; }

double s2moe_unique_expert_bytes(const s2moe_ctx *ctx, int32_t n_unique)
{
    if (!ctx) return 0.0;
    const Shape &sh = ctx->shape;
    auto mat = [&](int rows, int K) {
        double b = (double)rows * (double)row_bytes(sh.weight_dtype, K);
        if (sh.weight_dtype == DT_Q4B32) b += (double)rows * (K / 32) * 2.0;
        return b;
    };
    const double routed = 2.0 * mat(sh.f, sh.d) + mat(sh.d, sh.f);
    const double shared = sh.n_sh ? sh.n_sh * (2.0 * mat(sh.f_sh, sh.d) + mat(sh.d, sh.f_sh)) : 0.0;
    return (double)n_unique * routed + shared;
}

int s2moe_profile_begin(s2moe_ctx *ctx, int32_t max_records)
{
    if (!ctx || max_records < 0) return S2MOE_EINVAL;
    while (ctx->prof_ev.size() < 2 * (size_t)max_records) {
        cudaEvent_t ev;
        CU(ctx, cudaEventCreate(&ev));
        ctx->prof_ev.push_back(ev);
    }
    ctx->prof_cap = (size_t)max_records;
    ctx->prof_cls.clear();
    ctx->prof_on = true;
    return S2MOE_OK;
}

int s2moe_profile_end(s2moe_ctx *ctx, int32_t n_classes, double *ms_out, int64_t *launches_out)
{
    if (!ctx || !ms_out || !launches_out || n_classes < 1) return S2MOE_EINVAL;
    ctx->prof_on = false;
    CU(ctx, cudaDeviceSynchronize());
    for (int c = 0; c < n_classes; ++c) { ms_out[c] = 0.0; launches_out[c] = 0; }
    for (size_t r = 0; r < ctx->prof_cls.size(); ++r) {
        float ms = 0.f;
        CU(ctx, cudaEventElapsedTime(&ms, ctx->prof_ev[2 * r], ctx->prof_ev[2 * r + 1]));
        const int c = ctx->prof_cls[r];
        if (c < n_classes) { ms_out[c] += ms; launches_out[c] += 1; }
    }
    ctx->prof_cls.clear();
    return S2MOE_OK;
}

const char *s2moe_kernel_class_name(int32_t cls)
{
    switch (cls) {
        case KC_ROUTER: return "route_kernel";
        case KC_GATING: return "(unused)";
        case KC_GATEUP: return "ffn_gateup_simple";
        case KC_DOWN: return "ffn_down_simple";
        case KC_STREAM: return "ffn_stream_kernel";
        case KC_TC: return "ffn_tc_kernel";
        case KC_LAYER: return "layer_tc_kernel";
        default: return nullptr;
    }
}

int s2moe_debug_read(s2moe_ctx *ctx, int32_t what, void *host_out, size_t bytes)
{
    if (!ctx || !host_out) return S2MOE_EINVAL;
    CU(ctx, cudaDeviceSynchronize());
    int32_t hdr[4];
    CU(ctx, cudaMemcpy(hdr, ctx->ws.header, sizeof(hdr), cudaMemcpyDeviceToHost));
    const Shape &sh = ctx->shape;
    const int G = sh.E + sh.n_sh, B = ctx->last_B;
    const void *src = nullptr;
    size_t need = 0;
    switch (what) {
        case 0: src = ctx->ws.logits; need = sizeof(double) * (size_t)B * sh.E; break;
        case 1: src = ctx->ws.counts; need = 4 * (size_t)G; break;
        case 2: src = ctx->ws.offsets; need = 4 * (size_t)(G + 1); break;
        case 3: src = ctx->ws.slot_token; need = 4 * (size_t)hdr[1]; break;
        case 4: src = ctx->ws.slot_w; need = 4 * (size_t)hdr[1]; break;
        case 5: src = ctx->ws.active; need = 4 * (size_t)hdr[0]; break;
        case 6: src = ctx->ws.header; need = 16; break;
        case 7: src = ctx->ws.header + 8; need = 32; break;
        case 8: src = ctx->ws.act; need = bytes; break;   // timing build: per-warp cycle counters
        default: return S2MOE_EINVAL;
    }
    if (bytes < need) return S2MOE_EINVAL;
    CU(ctx, cudaMemcpy(host_out, src, need, cudaMemcpyDeviceToHost));
    return S2MOE_OK;
}

// ---- routing without allocation -------------------------------------------------------

namespace {

// Scratch of s2moe_route_noalloc.  In host code this name is only a handle for
// cudaGetSymbolAddress; kernels get the device address that call returns.
static __device__ __align__(256) unsigned char g_noalloc_scratch[S2MOE_NOALLOC_SCRATCH_BYTES];

constexpr int kNoallocMaxDevices = 64;
void *g_noalloc_ptr[kNoallocMaxDevices] = {};

__global__ void noalloc_gate_out_kernel(const double *__restrict__ gate_logit, float *__restrict__ gate_out, int B)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) gate_out[b] = (float)(1.0 / (1.0 + exp(-gate_logit[b])));
}

}  // namespace

int s2moe_route_noalloc(const s2moe_config *cfg, int32_t n_tokens, const void *router, const void *gate_vec,
                        const void *hidden, const float *conf, int32_t *sel_idx, float *sel_w,
                        int32_t *n_unique, float *gate_out, void *cuda_stream)
{
    if (!cfg || !router || !hidden || !sel_idx || !sel_w || !n_unique) return S2MOE_EINVAL;
    if (cfg->d_model < 64 || cfg->d_model % 64) return S2MOE_EINVAL;
    if (cfg->n_experts < 1 || cfg->top_k < 1 || cfg->top_k > cfg->n_experts || cfg->top_k > S2MOE_MAX_TOP_K)
        return S2MOE_EINVAL;
    if (cfg->act_dtype != S2MOE_F32 && cfg->act_dtype != S2MOE_BF16) return S2MOE_EINVAL;
    if (cfg->router_dtype != S2MOE_F32 && cfg->router_dtype != S2MOE_BF16) return S2MOE_EINVAL;
    if ((cfg->renorm != 0 && cfg->renorm != 1) || (cfg->weight_mode != 0 && cfg->weight_mode != 1)) return S2MOE_EINVAL;
    if (cfg->cap < cfg->top_k || cfg->cap > cfg->n_experts || !(cfg->alpha >= 0.0f)) return S2MOE_EINVAL;
    if (!aligned16(router) || !aligned16(hidden) || (gate_vec && !aligned16(gate_vec))) return S2MOE_EINVAL;
    if (n_tokens < 0 || n_tokens > S2MOE_NOALLOC_MAX_TOKENS || cfg->n_experts > S2MOE_NOALLOC_MAX_EXPERTS)
        return S2MOE_ERANGE;
    if (n_tokens == 0) return S2MOE_OK;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    // once per device: the scratch array's device address, and the kernels' shared-memory limit
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoallocMaxDevices) return S2MOE_ECUDA;
    if (!g_noalloc_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return S2MOE_ECUDA;
        if (prepare_route() != cudaSuccess) return S2MOE_ECUDA;
        // load the small kernel's module now as well, so that no later call (one made under a
        // stream capture, say) is the first to touch it
        cudaFuncAttributes fa;
        if (cudaFuncGetAttributes(&fa, noalloc_gate_out_kernel) != cudaSuccess) return S2MOE_ECUDA;
        g_noalloc_ptr[dev] = p;
    }
    uint8_t *base = (uint8_t *)g_noalloc_ptr[dev];

    // carve the scratch: the routing kernel's workspace for E <= 128 experts, B <= 64 tokens
    const int T = S2MOE_NOALLOC_MAX_TOKENS, E = S2MOE_NOALLOC_MAX_EXPERTS, K = S2MOE_MAX_TOP_K;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    Workspace ws{};
    ws.logits = (double *)(base + take(sizeof(double) * T * E));
    ws.gate_logit = (double *)(base + take(sizeof(double) * T));
    uint8_t *zero_begin = base + off;                       // words that must start at zero
    ws.ticket = (unsigned int *)(base + take(256));
    ws.status = (int32_t *)(base + take(256));
    uint8_t *zero_end = base + off;
    ws.header = (int32_t *)(base + take(256));
    ws.counts = (int32_t *)(base + take(4 * (size_t)E));
    ws.offsets = (int32_t *)(base + take(4 * (size_t)(E + 1)));
    ws.slot_token = (int32_t *)(base + take(4 * (size_t)T * K));
    ws.slot_w = (float *)(base + take(4 * (size_t)T * K));
    ws.active = (int32_t *)(base + take(4 * (size_t)E));
    ws.tokmask = (unsigned long long *)(base + take(8 * (size_t)E));
    static_assert(sizeof(double) * S2MOE_NOALLOC_MAX_TOKENS * S2MOE_NOALLOC_MAX_EXPERTS + 24 * 1024 <=
                      S2MOE_NOALLOC_SCRATCH_BYTES, "scratch too small");
    if (off > S2MOE_NOALLOC_SCRATCH_BYTES) return S2MOE_ERANGE;

    Shape sh{};
    sh.d = cfg->d_model; sh.f = 0; sh.E = cfg->n_experts; sh.k = cfg->top_k; sh.n_sh = 0; sh.f_sh = 0;
    sh.act_dtype = cfg->act_dtype; sh.router_dtype = cfg->router_dtype; sh.weight_dtype = DT_BF16;
    sh.renorm = cfg->renorm; sh.cap = cfg->cap; sh.weight_mode = cfg->weight_mode; sh.plan = 1; sh.op_cap = 0;
    sh.alpha = (double)cfg->alpha;
    if (cudaMemsetAsync(zero_begin, 0, (size_t)(zero_end - zero_begin), st) != cudaSuccess) return S2MOE_ECUDA;
    const int rows = sh.E + (gate_vec ? 1 : 0);
    const size_t smem = route_smem(n_tokens, sh.E);
    const bool af = sh.act_dtype == DT_F32, rf = sh.router_dtype == DT_F32;
    // (the no-allocation entry covers up to 128 experts: two or four per lane in the gating)
#define S2MOE_ROUTE_NA(A, R)                                                                                         \
    do {                                                                                                             \
        if (sh.E <= 64)                                                                                              \
            route_kernel<A, R, 2><<<rows, kRouteThreads, smem, st>>>(sh, n_tokens, ws, hidden, router, gate_vec, conf, \
                                                                     sel_idx, sel_w, n_unique, ZeroList{});          \
        else                                                                                                         \
            route_kernel<A, R, 4><<<rows, kRouteThreads, smem, st>>>(sh, n_tokens, ws, hidden, router, gate_vec, conf, \
                                                                     sel_idx, sel_w, n_unique, ZeroList{});          \
    } while (0)
    if (af && rf) S2MOE_ROUTE_NA(DT_F32, DT_F32);
    else if (af) S2MOE_ROUTE_NA(DT_F32, DT_BF16);
    else if (rf) S2MOE_ROUTE_NA(DT_BF16, DT_F32);
    else S2MOE_ROUTE_NA(DT_BF16, DT_BF16);
#undef S2MOE_ROUTE_NA
    if (gate_vec && gate_out) noalloc_gate_out_kernel<<<1, 64, 0, st>>>(ws.gate_logit, gate_out, n_tokens);
    return cudaGetLastError() == cudaSuccess ? S2MOE_OK : S2MOE_ECUDA;
}

int s2moe_route_noalloc_status(int32_t *host_out)
{
    if (!host_out) return S2MOE_EINVAL;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoallocMaxDevices) return S2MOE_ECUDA;
    *host_out = 0;
    if (!g_noalloc_ptr[dev]) return S2MOE_OK;            // never called on this device: nothing to report
    if (cudaDeviceSynchronize() != cudaSuccess) return S2MOE_ECUDA;
    // the status word sits behind the logits, the gate logits and the arrival words (see the carving above)
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    take(sizeof(double) * S2MOE_NOALLOC_MAX_TOKENS * S2MOE_NOALLOC_MAX_EXPERTS);
    take(sizeof(double) * S2MOE_NOALLOC_MAX_TOKENS);
    take(256);
    const size_t o_status = take(256);
    if (cudaMemcpy(host_out, (const uint8_t *)g_noalloc_ptr[dev] + o_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess)
        return S2MOE_ECUDA;
    return *host_out != 0 ? S2MOE_ETIMEOUT : S2MOE_OK;
}

// ---- routing-aware adaptive expansion (no context, no allocation) ----------------------

int s2moe_expert_masks(const int32_t *sel_idx, int32_t n_tokens, int32_t top_k, int32_t n_experts, uint64_t *masks,
                       int32_t stride_words, void *cuda_stream)
{
    if (n_tokens < 0 || top_k < 1 || top_k > S2MOE_MAX_TOP_K || n_experts < 1 || n_experts > S2MOE_MAX_EXPERTS)
        return S2MOE_EINVAL;
    const int words = (n_experts + 63) / 64;
    if (stride_words < words) return S2MOE_EINVAL;
    if (n_tokens == 0) return S2MOE_OK;
    if (!sel_idx || !masks) return S2MOE_EINVAL;
    expert_masks_kernel<<<(n_tokens + 127) / 128, 128, 0, (cudaStream_t)cuda_stream>>>(
        sel_idx, n_tokens, top_k, words, reinterpret_cast<unsigned long long *>(masks), stride_words);
    return cudaGetLastError() == cudaSuccess ? S2MOE_OK : S2MOE_ECUDA;
}

int s2moe_adaptive_expand(int32_t n_cand, int32_t n_layers, int32_t n_experts, const int32_t *parent,
                          const float *p_tok, const uint64_t *masks, const float *c_draft, float t_ar, float t_exp,
                          int32_t *admitted, int32_t *order, int32_t *n_admitted, uint64_t *union_out,
                          void *cuda_stream)
{
    if (n_cand < 1 || n_layers < 1 || n_experts < 1 || n_experts > S2MOE_MAX_EXPERTS) return S2MOE_EINVAL;
    if (!parent || !p_tok || !masks || !admitted || !order || !n_admitted) return S2MOE_EINVAL;
    const int lw = n_layers * ((n_experts + 63) / 64);
    if (n_cand > kExpandMaxCand || lw > kExpandMaxWords) return S2MOE_ERANGE;
    const int threads = ((n_cand + 31) / 32) * 32;
    adaptive_expand_kernel<<<1, threads, 0, (cudaStream_t)cuda_stream>>>(
        n_cand, lw, parent, p_tok, reinterpret_cast<const unsigned long long *>(masks), c_draft, t_ar, t_exp,
        admitted, order, n_admitted, reinterpret_cast<unsigned long long *>(union_out));
    return cudaGetLastError() == cudaSuccess ? S2MOE_OK : S2MOE_ECUDA;
}

}  // extern "C"
