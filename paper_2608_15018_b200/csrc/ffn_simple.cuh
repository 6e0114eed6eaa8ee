// Plain CUDA-core expert kernels (kernel plan 1): every storage format, one warp per
// weight row, fp32 accumulation.  They read each selected expert's weights from HBM
// once (further token chunks of the same row hit L1/L2) and serve as the fp32 path
// and as an independent check of the streaming kernels.
//
//   ffn_gateup_simple : a[slot][j] = silu(W_g[e][j] . x) * (W_u[e][j] . x)
//   ffn_down_simple   : y[token][r] += p * (W_d[e][r] . a[slot])
#pragma once

#include "common.cuh"

namespace s2moe {

constexpr int kSimpleWarps = 8;
constexpr int kSimpleTokChunk = 8;    // tokens staged in shared memory at a time
constexpr int kSimpleKChunk = 2048;   // contraction elements staged at a time

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

struct GroupView {
    const uint8_t *gate, *up, *down;        // first row of this group's matrices
    const uint8_t *sgate, *sup, *sdown;     // first scale
    int f;                                  // inner dim of this group
    int count, offset;                      // tokens, first slot
};

__device__ __forceinline__ GroupView group_view(const Shape &sh, const LayerPtrs &lp, const Workspace &ws,
                                                int group)
{
    GroupView g;
    const int wt = sh.weight_dtype;
    if (group < sh.E) {
        g.f = sh.f;
        const size_t gu = (size_t)group * sh.f, dn = (size_t)group * sh.d;
        g.gate = (const uint8_t *)lp.w_gate + gu * row_bytes(wt, sh.d);
        g.up = (const uint8_t *)lp.w_up + gu * row_bytes(wt, sh.d);
        g.down = (const uint8_t *)lp.w_down + dn * row_bytes(wt, sh.f);
        g.sgate = (const uint8_t *)lp.s_gate + gu * (sh.d / 32) * 2;
        g.sup = (const uint8_t *)lp.s_up + gu * (sh.d / 32) * 2;
        g.sdown = (const uint8_t *)lp.s_down + dn * (sh.f / 32) * 2;
    } else {
        const int s = group - sh.E;
        g.f = sh.f_sh;
        const size_t gu = (size_t)s * sh.f_sh, dn = (size_t)s * sh.d;
        g.gate = (const uint8_t *)lp.sh_gate + gu * row_bytes(wt, sh.d);
        g.up = (const uint8_t *)lp.sh_up + gu * row_bytes(wt, sh.d);
        g.down = (const uint8_t *)lp.sh_down + dn * row_bytes(wt, sh.f_sh);
        g.sgate = (const uint8_t *)lp.sh_s_gate + gu * (sh.d / 32) * 2;
        g.sup = (const uint8_t *)lp.sh_s_up + gu * (sh.d / 32) * 2;
        g.sdown = (const uint8_t *)lp.sh_s_down + dn * (sh.f_sh / 32) * 2;
    }
    g.count = ws.counts[group];
    g.offset = ws.offsets[group];
    return g;
}

// grid (ceil(max(f, f_sh) / kSimpleWarps), E + n_sh); dynamic smem kSimpleTokChunk*kSimpleKChunk floats
template <int WT, int ACT>
__global__ void __launch_bounds__(kSimpleWarps * 32)
ffn_gateup_simple(Shape sh, LayerPtrs lp, Workspace ws, const void *__restrict__ hidden)
{
    extern __shared__ float s_x[];  // [tok chunk][k chunk]
    if ((int)blockIdx.y >= ws.header[0]) return;
    const int group = ws.active[blockIdx.y];
    const GroupView g = group_view(sh, lp, ws, group);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x * kSimpleWarps + warp;
    if (blockIdx.x * kSimpleWarps >= g.f) return;
    const int d = sh.d, n_routed = ws.header[3] * sh.k;
    const size_t ab = ACT == DT_F32 ? 4 : 2;
    const bool row_ok = j < g.f;
    const uint8_t *grow = g.gate + (size_t)j * row_bytes(WT, d);
    const uint8_t *urow = g.up + (size_t)j * row_bytes(WT, d);
    const uint8_t *gs = g.sgate + (size_t)j * (d / 32) * 2;
    const uint8_t *us = g.sup + (size_t)j * (d / 32) * 2;

    for (int t0 = 0; t0 < g.count; t0 += kSimpleTokChunk) {
        const int nt = min(kSimpleTokChunk, g.count - t0);
        float ag[kSimpleTokChunk], au[kSimpleTokChunk];
#pragma unroll
        for (int t = 0; t < kSimpleTokChunk; ++t) ag[t] = au[t] = 0.f;
        for (int k0 = 0; k0 < d; k0 += kSimpleKChunk) {
            const int kc = min(kSimpleKChunk, d - k0);
            __syncthreads();
            for (int i = threadIdx.x * 8; i < nt * kc; i += blockDim.x * 8) {
                const int t = i / kc, c = i - t * kc;
                const int tok = ws.slot_token[g.offset + t0 + t];
                float v[8];
                load8_plain<ACT>((const uint8_t *)hidden + (size_t)tok * d * ab, k0 + c, v);
#pragma unroll
                for (int q = 0; q < 8; ++q) s_x[t * kSimpleKChunk + c + q] = v[q];
            }
            __syncthreads();
            if (row_ok) {
                for (int c = lane * 8; c < kc; c += 256) {
                    float wg[8], wu[8];
                    load8_weight<WT>(grow, gs, k0 + c, wg);
                    load8_weight<WT>(urow, us, k0 + c, wu);
#pragma unroll
                    for (int t = 0; t < kSimpleTokChunk; ++t) {
                        if (t < nt) {
                            const float4 x0 = *reinterpret_cast<const float4 *>(&s_x[t * kSimpleKChunk + c]);
                            const float4 x1 = *reinterpret_cast<const float4 *>(&s_x[t * kSimpleKChunk + c + 4]);
                            ag[t] += wg[0] * x0.x + wg[1] * x0.y + wg[2] * x0.z + wg[3] * x0.w +
                                     wg[4] * x1.x + wg[5] * x1.y + wg[6] * x1.z + wg[7] * x1.w;
                            au[t] += wu[0] * x0.x + wu[1] * x0.y + wu[2] * x0.z + wu[3] * x0.w +
                                     wu[4] * x1.x + wu[5] * x1.y + wu[6] * x1.z + wu[7] * x1.w;
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int t = 0; t < kSimpleTokChunk; ++t) {
            if (t < nt) {
                const float sg = warp_sum_f(ag[t]), su = warp_sum_f(au[t]);
                if (lane == 0 && row_ok) {
                    const int slot = g.offset + t0 + t;
                    ws.act[act_offset(slot, n_routed, sh.f, sh.f_sh) + j] = silu_mul(sg, su);
                }
            }
        }
    }
}

// grid (ceil(d / kSimpleWarps), E + n_sh); same dynamic smem
template <int WT>
__global__ void __launch_bounds__(kSimpleWarps * 32)
ffn_down_simple(Shape sh, LayerPtrs lp, Workspace ws, float *__restrict__ y)
{
    extern __shared__ float s_x[];
    if ((int)blockIdx.y >= ws.header[0]) return;
    const int group = ws.active[blockIdx.y];
    const GroupView g = group_view(sh, lp, ws, group);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = blockIdx.x * kSimpleWarps + warp;
    const int d = sh.d, f = g.f, n_routed = ws.header[3] * sh.k;
    const bool row_ok = r < d;
    const uint8_t *drow = g.down + (size_t)r * row_bytes(WT, f);
    const uint8_t *ds = g.sdown + (size_t)r * (f / 32) * 2;

    for (int t0 = 0; t0 < g.count; t0 += kSimpleTokChunk) {
        const int nt = min(kSimpleTokChunk, g.count - t0);
        float acc[kSimpleTokChunk];
#pragma unroll
        for (int t = 0; t < kSimpleTokChunk; ++t) acc[t] = 0.f;
        for (int k0 = 0; k0 < f; k0 += kSimpleKChunk) {
            const int kc = min(kSimpleKChunk, f - k0);
            __syncthreads();
            for (int i = threadIdx.x * 4; i < nt * kc; i += blockDim.x * 4) {
                const int t = i / kc, c = i - t * kc;
                const int slot = g.offset + t0 + t;
                const float4 v = *reinterpret_cast<const float4 *>(
                    &ws.act[act_offset(slot, n_routed, sh.f, sh.f_sh) + k0 + c]);
                *reinterpret_cast<float4 *>(&s_x[t * kSimpleKChunk + c]) = v;
            }
            __syncthreads();
            if (row_ok) {
                for (int c = lane * 8; c < kc; c += 256) {
                    float w[8];
                    load8_weight<WT>(drow, ds, k0 + c, w);
#pragma unroll
                    for (int t = 0; t < kSimpleTokChunk; ++t) {
                        if (t < nt) {
                            const float4 x0 = *reinterpret_cast<const float4 *>(&s_x[t * kSimpleKChunk + c]);
                            const float4 x1 = *reinterpret_cast<const float4 *>(&s_x[t * kSimpleKChunk + c + 4]);
                            acc[t] += w[0] * x0.x + w[1] * x0.y + w[2] * x0.z + w[3] * x0.w +
                                      w[4] * x1.x + w[5] * x1.y + w[6] * x1.z + w[7] * x1.w;
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int t = 0; t < kSimpleTokChunk; ++t) {
            if (t < nt) {
                const float s = warp_sum_f(acc[t]);
                if (lane == 0 && row_ok) {
                    const int slot = g.offset + t0 + t;
                    atomicAdd(&y[(size_t)ws.slot_token[slot] * d + r], ws.slot_w[slot] * s);
                }
            }
        }
    }
}

}  // namespace s2moe
