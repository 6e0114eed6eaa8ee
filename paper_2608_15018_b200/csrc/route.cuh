// Router logits and reuse-aware expert gating (Sec. 4.2) for one draft batch.
//
//   route_kernel : l_{b,e} = h_b . W_r[e] (and the shared-expert gate logit) in float64, so
//                  that the discrete choices below do not depend on the summation order;
//                  the last block to finish then runs gating_block:
//   gating_block : Eq. 4 aggregation, TopCap, lambda_b, biased top-k, mixing weights,
//                  union / unique count, token->expert bucketing, stage tables.
#pragma once

#include "common.cuh"
#include "ffn_stream.cuh"

namespace s2moe {


__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// order (value descending, id ascending): is a before b?
__device__ __forceinline__ bool before1(double va, int a, double vb, int b)
{
    return (va > vb) | ((va == vb) & (a < b));
}
// order (l' descending, l descending, id ascending)
__device__ __forceinline__ bool before2(double l2a, double la, int a, double l2b, double lb, int b)
{
    return (l2a > l2b) | ((l2a == l2b) & ((la > lb) | ((la == lb) & (a < b))));
}

// Gating of one batch by one thread block (any block size that is a multiple of 32).
// s_l: shared memory for B*E doubles (the logits, copied from the workspace).
__device__ __forceinline__ void gating_block(const Shape &sh, int B, const Workspace &ws, const float *__restrict__ conf,
                                             int has_gate, int32_t *__restrict__ sel_idx, float *__restrict__ sel_w,
                                             int32_t *__restrict__ n_unique, double *s_l)
{
    __shared__ double s_g[kMaxExperts];
    __shared__ unsigned char s_star[kMaxExperts];
    __shared__ double s_w[kMaxTokens], s_top1[kMaxTokens], s_kth[kMaxTokens], s_lam[kMaxTokens];
    __shared__ int s_sel[kMaxTokens * kMaxTopK];
    __shared__ float s_pw[kMaxTokens * kMaxTopK];
    __shared__ unsigned long long s_mask[kMaxExperts];
    __shared__ int s_cnt[kMaxExperts], s_off[kMaxExperts + 1], s_pos[kMaxExperts];
    __shared__ int s_U;

    const int tid = threadIdx.x, nt = blockDim.x;
    const int E = sh.E, k = sh.k, cap = sh.cap;
    const bool bias_on = sh.alpha > 0.0 && cap < E && k < E;
#ifdef S2MOE_TIMING
    long long *tm = reinterpret_cast<long long *>(ws.act) + 148 * 64;
    int tmi = 0;
#define GATE_MARK() do { __syncthreads(); if (tid == 0) tm[tmi] = clock64(); ++tmi; } while (0)
#else
#define GATE_MARK() do { } while (0)
#endif
    GATE_MARK();

    for (int i = tid; i < B * E; i += nt) s_l[i] = __ldcg(&ws.logits[i]);
    for (int b = tid; b < B; b += nt) {
        s_w[b] = conf ? (double)conf[b] : 1.0;
        s_lam[b] = 0.0;
    }
    for (int e = tid; e < E; e += nt) { s_star[e] = 0; s_mask[e] = 0ull; }
    __syncthreads();

    GATE_MARK();
    if (bias_on) {
        // Eq. 4: g_e = sum_b w_b l_{b,e}, tokens in ascending order
        for (int e = tid; e < E; e += nt) {
            double g = 0.0;
            for (int b = 0; b < B; ++b) g = fma(s_w[b], s_l[b * E + e], g);
            s_g[e] = g;
        }
        __syncthreads();
        // TopCap by rank
        for (int e = tid; e < E; e += nt) {
            int rank = 0;
            const double ge = s_g[e];
#pragma unroll 8
            for (int o = 0; o < E; ++o) rank += before1(s_g[o], o, ge, e);
            s_star[e] = rank < cap;
        }
        // order statistics of the original logits: top-1 and (k+1)-th
        for (int i = tid; i < B * E; i += nt) {
            const int b = i / E, e = i - b * E;
            const double le = s_l[i];
            int rank = 0;
#pragma unroll 8
            for (int o = 0; o < E; ++o) rank += before1(s_l[b * E + o], o, le, e);
            if (rank == 0) s_top1[b] = le;
            if (rank == k) s_kth[b] = le;
        }
        __syncthreads();
        for (int b = tid; b < B; b += nt) s_lam[b] = sh.alpha * (s_top1[b] - s_kth[b]);
        __syncthreads();
    }

    GATE_MARK();
    // biased top-k by rank
    for (int i = tid; i < B * E; i += nt) {
        const int b = i / E, e = i - b * E;
        const double lam = s_lam[b];
        const double le = s_l[i];
        const double l2e = s_star[e] ? le + lam : le;
        int rank = 0;
#pragma unroll 8
        for (int o = 0; o < E; ++o) {
            const double lo = s_l[b * E + o];
            const double l2o = s_star[o] ? lo + lam : lo;
            rank += before2(l2o, lo, o, l2e, le, e);
        }
        if (rank < k) s_sel[b * k + rank] = e;
    }
    __syncthreads();

    GATE_MARK();
    // mixing weights: one warp per token
    {
        const int warp = tid >> 5, lane = tid & 31, nw = nt >> 5;
        for (int b = warp; b < B; b += nw) {
            const double lam = sh.weight_mode ? s_lam[b] : 0.0;
            double zmax = -1.0e300;
            for (int e = lane; e < E; e += 32) {
                const double z = s_l[b * E + e] + (s_star[e] ? lam : 0.0);
                zmax = fmax(zmax, z);
            }
            zmax = warp_max(zmax);
            double den = 0.0;
            for (int e = lane; e < E; e += 32) {
                const double z = s_l[b * E + e] + (s_star[e] ? lam : 0.0);
                den += exp(z - zmax);
            }
            den = warp_sum(den);
            double p = 0.0;
            int e = 0;
            if (lane < k) {
                e = s_sel[b * k + lane];
                const double z = s_l[b * E + e] + (s_star[e] ? lam : 0.0);
                p = exp(z - zmax) / den;
            }
            if (sh.renorm) {
                const double tot = warp_sum(p);
                p /= tot;
            }
            if (lane < k) {
                s_pw[b * k + lane] = (float)p;
                sel_idx[b * k + lane] = e;
                sel_w[b * k + lane] = (float)p;
                atomicOr(&s_mask[e], 1ull << b);
            }
        }
    }
    __syncthreads();

    GATE_MARK();
    // union, unique count, exclusive scan, list of active experts
    for (int e = tid; e < E; e += nt) s_cnt[e] = __popcll(s_mask[e]);
    __syncthreads();
    for (int e = tid; e < E; e += nt) {
        int off = 0, pos = 0;
#pragma unroll 8
        for (int o = 0; o < e; ++o) { off += s_cnt[o]; pos += s_cnt[o] > 0; }
        s_off[e] = off;
        s_pos[e] = pos;
        if (e == E - 1) { s_off[E] = off + s_cnt[e]; s_U = pos + (s_cnt[e] > 0); }
    }
    __syncthreads();
    const int U = s_U, n_routed = B * k;
    for (int e = tid; e < E; e += nt) {
        ws.counts[e] = s_cnt[e];
        ws.offsets[e] = s_off[e];
        if (s_cnt[e] > 0) ws.active[s_pos[e]] = e;
    }
    // bucket the (token, choice) pairs: tokens ascending inside an expert
    for (int i = tid; i < n_routed; i += nt) {
        const int b = i / k;
        const int e = s_sel[i];
        const int pos = s_off[e] + __popcll(s_mask[e] & ((1ull << b) - 1ull));
        ws.slot_token[pos] = b;
        ws.slot_w[pos] = s_pw[i];
    }
    // shared experts: every token, weight c_b
    for (int i = tid; i < sh.n_sh * B; i += nt) {
        const int s = i / B, b = i - s * B;
        float c = 1.0f;
        if (has_gate) c = (float)(1.0 / (1.0 + exp(-__ldcg(&ws.gate_logit[b]))));
        ws.slot_token[n_routed + i] = b;
        ws.slot_w[n_routed + i] = c;
        if (b == 0) {
            ws.counts[E + s] = B;
            ws.offsets[E + s] = n_routed + s * B;
            ws.active[U + s] = E + s;
        }
    }
    GATE_MARK();
    for (int e = tid; e < E; e += nt) ws.tokmask[e] = s_mask[e];
    for (int s = tid; s < sh.n_sh; s += nt) ws.tokmask[E + s] = B >= 64 ? ~0ull : ((1ull << B) - 1ull);
    if (sh.plan == 2) {
        // stage tables of the streaming kernel: per active group, its first phase-1 stage
        // (4 gate + 4 up rows each) and first phase-2 stage (8 down rows x one K-slice)
        __syncthreads();
        for (int e = tid; e < E; e += nt)
            s_cnt[e] = s_cnt[e] > 0 ? st_nks(sh.f, s_cnt[e], sh.op_cap, sh.d) * (sh.d / 8) : 0;   // phase-2 stages
        __syncthreads();
        for (int e = tid; e < E; e += nt) {
            if (s_mask[e]) {
                int pre = 0;
                for (int o = 0; o < e; ++o) pre += s_cnt[o];
                const int a = s_pos[e];
                ws.upfx1[a] = a * (sh.f / 4);
                ws.upfx2[a] = pre;
                ws.sync[a] = 0;
                if (a == U - 1) s_off[0] = pre + s_cnt[e];   // all routed phase-2 stages
            }
        }
        __syncthreads();
        if (tid == 0) {
            int t1 = U * (sh.f / 4), t2 = s_off[0];
            for (int s = 0; s <= sh.n_sh; ++s) {
                ws.upfx1[U + s] = t1;
                ws.upfx2[U + s] = t2;
                ws.sync[U + s] = 0;
                if (s < sh.n_sh) {
                    t1 += sh.f_sh / 4;
                    t2 += st_nks(sh.f_sh, B, sh.op_cap, sh.d) * (sh.d / 8);
                }
            }
            ws.header[4] = t1;
            ws.header[5] = t2;
        }
    }
    GATE_MARK();
    if (tid == 0) {
        ws.offsets[E + sh.n_sh] = n_routed + sh.n_sh * B;
        ws.header[0] = U + sh.n_sh;
        ws.header[1] = n_routed + sh.n_sh * B;
        ws.header[2] = U;
        ws.header[3] = B;
        *n_unique = U;
    }
}

// 4 consecutive elements of a plain (f32 / bf16) row starting at column c (c % 4 == 0)
template <int DT>
__device__ __forceinline__ void load4_plain(const void *row, int c, float (&v)[4])
{
    if (DT == DT_F32) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(row) + c));
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    } else {
        const uint2 a = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const uint16_t *>(row) + c));
        v[0] = bf16_lo(a.x); v[1] = bf16_hi(a.x); v[2] = bf16_lo(a.y); v[3] = bf16_hi(a.y);
    }
}

constexpr int kRouteThreads = 512;
constexpr int kRouteTok = 16;   // tokens accumulated per pass

// Router logits and gating in one launch.  Block r computes row r of the router (row E is the
// shared-expert gate vector) against all B tokens in float64; the block that finishes last
// (atomic ticket, nobody waits) then runs the gating for the whole batch.
// Dynamic shared memory: max(B * E, 16 * kRouteTok) doubles.
template <int ACT, int RT>
__global__ void __launch_bounds__(kRouteThreads)
route_kernel(Shape sh, int B, Workspace ws, const void *__restrict__ hidden, const void *__restrict__ router,
             const void *__restrict__ sh_scale, const float *__restrict__ conf, int32_t *__restrict__ sel_idx,
             float *__restrict__ sel_w, int32_t *__restrict__ n_unique)
{
    extern __shared__ double s_dyn[];
    __shared__ int s_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef S2MOE_TIMING
    const long long t_start = clock64();
#endif
    const int row = blockIdx.x, d = sh.d;
    const size_t rb = RT == DT_F32 ? 4 : 2, ab = ACT == DT_F32 ? 4 : 2;
    const uint8_t *wrow = row < sh.E ? reinterpret_cast<const uint8_t *>(router) + (size_t)row * d * rb
                                     : reinterpret_cast<const uint8_t *>(sh_scale);
    for (int b0 = 0; b0 < B; b0 += kRouteTok) {
        double acc[kRouteTok];
#pragma unroll
        for (int t = 0; t < kRouteTok; ++t) acc[t] = 0.0;
        for (int c = tid * 4; c < d; c += kRouteThreads * 4) {
            float w[4];
            load4_plain<RT>(wrow, c, w);
#pragma unroll
            for (int t = 0; t < kRouteTok; ++t) {
                if (b0 + t < B) {
                    float x[4];
                    load4_plain<ACT>(reinterpret_cast<const uint8_t *>(hidden) + (size_t)(b0 + t) * d * ab, c, x);
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[t] = fma((double)w[i], (double)x[i], acc[t]);
                }
            }
        }
#pragma unroll
        for (int t = 0; t < kRouteTok; ++t) {
            if (b0 + t < B) {           // uniform across the block
                const double s = warp_sum(acc[t]);
                if (lane == 0) s_dyn[warp * kRouteTok + t] = s;
            }
        }
        __syncthreads();
        if (tid < kRouteTok && b0 + tid < B) {
            double s = 0.0;
            for (int w = 0; w < kRouteThreads / 32; ++w) s += s_dyn[w * kRouteTok + tid];
            if (row < sh.E) ws.logits[(size_t)(b0 + tid) * sh.E + row] = s;
            else ws.gate_logit[b0 + tid] = s;
        }
        __syncthreads();
    }
    // the block that arrives last sees every row (release by fence + ticket, acquire by fence)
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned t = atomicAdd(ws.ticket, 1u);
        s_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid == 0) *ws.ticket = 0u;
#ifdef S2MOE_TIMING
    if (tid == 0) { long long *tm = reinterpret_cast<long long *>(ws.act) + 148 * 64; tm[15] = t_start; tm[14] = clock64(); }
#endif
    gating_block(sh, B, ws, conf, sh_scale ? 1 : 0, sel_idx, sel_w, n_unique, s_dyn);
}

}  // namespace s2moe
