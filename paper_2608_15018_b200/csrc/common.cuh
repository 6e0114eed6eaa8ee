// Shared declarations of the sm_100a MoE verification library: limits, the
// workspace that the routing kernel fills and the expert kernels consume, and
// decoders of the three storage formats.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace s2moe {

constexpr int kMaxTokens = 64;
constexpr int kMaxExperts = 256;
constexpr int kMaxTopK = 16;
constexpr int kMaxShared = 4;

enum : int { DT_F32 = 0, DT_BF16 = 1, DT_Q4B32 = 2 };

// device status codes (non-zero: a bounded wait gave up)
enum : int { ST_OK = 0, ST_MBAR_TIMEOUT = 1, ST_DEP_TIMEOUT = 2, ST_TICKET_TIMEOUT = 3, ST_BAD_PLAN = 4 };

struct LayerPtrs {
    const void *router;
    const void *w_gate, *w_up, *w_down;
    const void *s_gate, *s_up, *s_down;
    const void *sh_gate, *sh_up, *sh_down;
    const void *sh_s_gate, *sh_s_up, *sh_s_down;
    const void *sh_scale;
};

// Problem shape, passed to kernels by value.
struct Shape {
    int d, f, E, k, n_sh, f_sh;
    int act_dtype, router_dtype, weight_dtype;
    int renorm, cap, weight_mode;
    int plan;              // 1: CUDA-core kernels, 2: streaming kernel (stage tables are built)
    int op_cap;            // streaming kernel: capacity of the phase-2 operand region, bytes
    double alpha;
};

// Device workspace.  "Groups" are the routed experts 0..E-1 followed by the shared
// experts E..E+n_sh-1; a "slot" is one (token, group) pair.  Slots are stored group
// by group, tokens ascending inside a group; routed slots come first (B*k of them).
struct Workspace {
    double *logits;        // [max_tokens][E]
    double *gate_logit;    // [max_tokens]  h_b . w_sg
    unsigned int *ticket;  // arrival counter of the routing kernel
    int32_t *status;       // device status word
    int32_t *header;       // {n_active, n_slots, U, B, ...}
    int32_t *counts;       // [E + n_sh] tokens per group
    int32_t *offsets;      // [E + n_sh + 1] first slot of each group
    int32_t *slot_token;   // [n_slots] token of each slot
    float *slot_w;         // [n_slots] mixing weight of each slot
    int32_t *active;       // [n_active] groups that have tokens, ascending
    float *act;            // SwiGLU activations: routed slot s at s*f, shared slot at
                           // B*k*f + (s - B*k)*f_sh
    int32_t *sync;         // streaming kernel: finished phase-1 stages per active group
    int32_t *upfx1;        // [n_active + 1] first phase-1 stage of each active group
    int32_t *upfx2;        // [n_active + 1] first phase-2 stage of each active group
    unsigned long long *tokmask;   // [E + n_sh] bit b set: token b is bucketed to the group
    uint4 *gtab;           // [n_active][2] {group, tokens, first slot, 0}, {mask lo, mask hi, 0, 0}: the
                           // active groups in their final form, or NULL when nobody reads it
    int32_t *early;        // 8 words of 64 bits, {tag << 32 | bits of 32 experts}: the experts whose first projection
                           // may start before the gating has ended, published by the routing kernel (see
                           // gating_block), or NULL
    const int32_t *slot_of;  // [E] device slot that holds each routed expert's weights (expert offloading), or
                             // NULL: every expert is resident at its own index
};

__device__ __forceinline__ size_t act_offset(int slot, int n_routed_slots, int f, int f_sh)
{
    return slot < n_routed_slots ? (size_t)slot * f
                                 : (size_t)n_routed_slots * f + (size_t)(slot - n_routed_slots) * f_sh;
}

// ---- decoding -------------------------------------------------------------

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// 8 consecutive elements of a plain (f32 / bf16) row starting at column c (c % 8 == 0)
template <int DT>
__device__ __forceinline__ void load8_plain(const void *row, int c, float (&v)[8])
{
    if (DT == DT_F32) {
        const float4 *p = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(row) + c);
        float4 a = __ldg(p), b = __ldg(p + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
        const uint4 *p = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(row) + c);
        uint4 a = __ldg(p);
        v[0] = bf16_lo(a.x); v[1] = bf16_hi(a.x); v[2] = bf16_lo(a.y); v[3] = bf16_hi(a.y);
        v[4] = bf16_lo(a.z); v[5] = bf16_hi(a.z); v[6] = bf16_lo(a.w); v[7] = bf16_hi(a.w);
    }
}

// 8 consecutive weights of a stored weight row (any weight format).  `row` points at
// the row's first byte, `srow` at the row's first scale (Q4B32 only).
template <int WT>
__device__ __forceinline__ void load8_weight(const void *row, const void *srow, int c, float (&v)[8])
{
    if (WT == DT_Q4B32) {
        uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(reinterpret_cast<const uint8_t *>(row) + c / 2));
        float s = __half2float(__ldg(reinterpret_cast<const __half *>(srow) + c / 32));
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (float)((int)((w >> (4 * i)) & 15u) - 8) * s;
    } else {
        load8_plain<WT>(row, c, v);
    }
}

// bytes of one weight row of K elements
__host__ __device__ __forceinline__ size_t row_bytes(int wt, int K)
{
    return wt == DT_F32 ? (size_t)K * 4 : wt == DT_BF16 ? (size_t)K * 2 : (size_t)K / 2;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return g / (1.0f + __expf(-g)) * u; }

}  // namespace s2moe
