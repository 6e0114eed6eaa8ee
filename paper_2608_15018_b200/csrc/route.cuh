// Router logits and reuse-aware expert gating (Sec. 4.2) for one draft batch.
//
//   route_kernel : l_{b,e} = h_b . W_r[e] (and the shared-expert gate logit) in float64, so
//                  that the discrete choices below do not depend on the summation order;
//                  block 0 then runs gating_block once every row has arrived:
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

// One copy of the double-precision exponential for the whole gating: the gating runs once, on
// one block, with a cold instruction cache, so its cost follows the amount of distinct code.
__device__ __noinline__ double exp_once(double x) { return exp(x); }

// Monotone map from doubles (no NaN) to unsigned integers: a < b  <=>  dkey(a) < dkey(b), and
// equal doubles (-0 included) have equal keys.  Keys of finite values are never 0.
__device__ __forceinline__ unsigned long long dkey(double x)
{
    const long long b = __double_as_longlong(x + 0.0);
    return (unsigned long long)(b ^ ((b >> 63) | (long long)0x8000000000000000ull));
}
__device__ __forceinline__ double dkey_value(unsigned long long k)
{
    const long long b = (long long)k;
    return __longlong_as_double(b < 0 ? (b ^ (long long)0x8000000000000000ull) : ~b);
}
// maximum of a 64-bit key over the warp: two 32-bit warp reductions
__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long k)
{
    const unsigned hi = (unsigned)(k >> 32);
    const unsigned mh = __reduce_max_sync(0xffffffffu, hi);
    const unsigned ml = __reduce_max_sync(0xffffffffu, hi == mh ? (unsigned)k : 0u);
    return ((unsigned long long)mh << 32) | ml;
}
// lanes (as a ballot) that hold the largest key among the lanes with `has`; the common case
// (one lane has the largest upper half) takes one warp reduction and one ballot
__device__ __forceinline__ unsigned warp_max_holders(unsigned long long k, bool has)
{
    const unsigned hi = has ? (unsigned)(k >> 32) : 0u;
    const unsigned mh = __reduce_max_sync(0xffffffffu, hi);
    bool hold = has && hi == mh;
    unsigned hb = __ballot_sync(0xffffffffu, hold);
    if (__popc(hb) > 1) {
        const unsigned ml = __reduce_max_sync(0xffffffffu, hold ? (unsigned)k : 0u);
        hold = hold && (unsigned)k == ml;
        hb = __ballot_sync(0xffffffffu, hold);
    }
    return hb;
}
__device__ __forceinline__ unsigned long long shfl_key(unsigned long long k, int src)
{
    const unsigned lo = __shfl_sync(0xffffffffu, (unsigned)k, src);
    const unsigned hi = __shfl_sync(0xffffffffu, (unsigned)(k >> 32), src);
    return ((unsigned long long)hi << 32) | lo;
}


// Order statistics of one token's original logits, one warp per token (lane owns experts lane,
// lane + 32, ...): lambda_b = alpha (l_(1) - l_(k+1)) by k + 1 rounds of a warp-wide maximum over
// integer keys, and, for weight_mode 0, the softmax denominator over the original logits.
template <int J>
__device__ __forceinline__ void gate_stats(const Shape &sh, int b, bool bias_on, const double *s_l, double *s_lam,
                                           double *s_zmax, double *s_den, int lane)
{
    const int E = sh.E, k = sh.k;
    unsigned long long k1[J];
    unsigned valid = 0;
#pragma unroll
    for (int j = 0; j < J; ++j) {
        const int e = lane + 32 * j;
        k1[j] = 0ull;
        if (e < E) { k1[j] = dkey(s_l[b * E + e]); valid |= 1u << j; }
    }
    unsigned long long top1 = 0ull, kth = 0ull;
    const int rounds = bias_on ? k + 1 : 1;
    if constexpr (J == 2) {
        // two elements per lane: the lane offers its larger one and, once that has won a round,
        // the other (a key of 0 = nothing left); a round is one reduction and one ballot
        unsigned long long cur = k1[0] > k1[1] ? k1[0] : k1[1], nxt = k1[0] > k1[1] ? k1[1] : k1[0];
#pragma unroll 1
        for (int r = 0; r < rounds; ++r) {
            const unsigned hb = warp_max_holders(cur, cur != 0ull);
            const int wl = __ffs(hb) - 1;
            if (r == 0) top1 = shfl_key(cur, wl);
            if (r == k) kth = shfl_key(cur, wl);
            if (lane == wl) { cur = nxt; nxt = 0ull; }       // drop one instance of the maximum
        }
    } else {
        unsigned alive = valid;
#pragma unroll 1
        for (int r = 0; r < rounds; ++r) {
            unsigned long long lm = 0ull;
            int bj = 0;
#pragma unroll
            for (int j = 0; j < J; ++j)
                if (((alive >> j) & 1u) && k1[j] > lm) { lm = k1[j]; bj = j; }
            const unsigned hb = warp_max_holders(lm, alive != 0u);
            const int wl = __ffs(hb) - 1;
            if (r == 0) top1 = shfl_key(lm, wl);
            if (r == k) kth = shfl_key(lm, wl);
            if (lane == wl) alive &= ~(1u << bj);            // drop one instance of the maximum
        }
    }
    const double ztop = dkey_value(top1);
    double den = 0.0;
    if (!sh.weight_mode) {
#pragma unroll 1
        for (int e = lane; e < E; e += 32) den += exp_once((s_l[b * E + e] + 0.0) - ztop);
        den = warp_sum(den);
    }
    if (lane == 0) {
        s_lam[b] = bias_on ? sh.alpha * (ztop - dkey_value(kth)) : 0.0;
        s_zmax[b] = ztop;
        s_den[b] = den;
    }
}

// Biased top-k of one token in the order (l' descending, l descending, id ascending), one
// winner per round, and the mixing weights of the winners.
template <int J>
__device__ __forceinline__ void gate_select(const Shape &sh, int b, const double *s_l, const unsigned char *s_star,
                                            const double *s_lam, const double *s_zmax, const double *s_den, int *s_sel,
                                            float *s_pw, unsigned long long *s_mask, int32_t *__restrict__ sel_idx,
                                            float *__restrict__ sel_w, int lane)
{
    const unsigned full = 0xffffffffu;
    const int E = sh.E, k = sh.k;
    const double lam = s_lam[b];
    double l[J];
    unsigned long long k1[J], k2[J];
    unsigned valid = 0, star = 0;
#pragma unroll
    for (int j = 0; j < J; ++j) {
        const int e = lane + 32 * j;
        l[j] = 0.0;
        k1[j] = 0ull;
        k2[j] = 0ull;
        if (e < E) {
            l[j] = s_l[b * E + e] + 0.0;
            k1[j] = dkey(l[j]);
            const unsigned st = s_star[e];
            star |= st << j;
            k2[j] = st ? dkey(l[j] + lam) : k1[j];
            valid |= 1u << j;
        }
    }
    if constexpr (J == 2) {
        // the lane offers its better element first (order: l' descending, l descending, id
        // ascending; element 0 has the lower id), then the other one
        const bool first0 = k2[0] > k2[1] || (k2[0] == k2[1] && k1[0] >= k1[1]);
        unsigned long long c2 = first0 ? k2[0] : k2[1], c1 = first0 ? k1[0] : k1[1];
        unsigned long long n2 = first0 ? k2[1] : k2[0], n1 = first0 ? k1[1] : k1[0];
        unsigned ce = (unsigned)lane + (first0 ? 0u : 32u), ne = (unsigned)lane + (first0 ? 32u : 0u);
#pragma unroll 1
        for (int r = 0; r < k; ++r) {
            unsigned hb = warp_max_holders(c2, c2 != 0ull);
            if (__popc(hb) > 1) {                       // equal biased logits: larger original logit first
                hb = warp_max_holders(c1, (hb >> lane) & 1u);
                if (__popc(hb) > 1) {                   // still equal: lower expert id first
                    const bool hold = (hb >> lane) & 1u;
                    const unsigned me = __reduce_min_sync(full, hold ? ce : 0xffffffffu);
                    hb = __ballot_sync(full, hold && ce == me);
                }
            }
            if (lane == __ffs(hb) - 1) {
                s_sel[b * k + r] = (int)ce;
                c2 = n2; c1 = n1; ce = ne;
                n2 = 0ull;
            }
        }
    } else {
        unsigned alive = valid;
#pragma unroll 1
        for (int r = 0; r < k; ++r) {
            unsigned long long b2 = 0ull, b1 = 0ull;
            int bj = -1;
#pragma unroll
            for (int j = 0; j < J; ++j) {
                if ((alive >> j) & 1u) {
                    const bool better = k2[j] > b2 || (k2[j] == b2 && k1[j] > b1);
                    if (bj < 0 || better) { b2 = k2[j]; b1 = k1[j]; bj = j; }
                }
            }
            const unsigned my_e = (unsigned)(lane + 32 * (bj < 0 ? 0 : bj));
            unsigned hb = warp_max_holders(b2, bj >= 0);
            if (__popc(hb) > 1) {                           // equal biased logits: larger original logit first
                hb = warp_max_holders(b1, (hb >> lane) & 1u);
                if (__popc(hb) > 1) {                       // still equal: lower expert id first
                    const bool hold = (hb >> lane) & 1u;
                    const unsigned me = __reduce_min_sync(full, hold ? my_e : 0xffffffffu);
                    hb = __ballot_sync(full, hold && my_e == me);
                }
            }
            if (lane == __ffs(hb) - 1) {
                alive &= ~(1u << bj);
                s_sel[b * k + r] = (int)my_e;
            }
        }
    }
    __syncwarp();
    // mixing weights: softmax over all experts of l (weight_mode 0) or l' (weight_mode 1)
    double zmax = s_zmax[b], den = s_den[b];
    const double lamw = sh.weight_mode ? lam : 0.0;
    if (sh.weight_mode) {
        unsigned long long zk = 0ull;
#pragma unroll
        for (int j = 0; j < J; ++j)
            if (((valid >> j) & 1u) && k2[j] > zk) zk = k2[j];
        zmax = dkey_value(warp_max_key(zk));
        den = 0.0;
#pragma unroll 1
        for (int e = lane; e < E; e += 32) den += exp_once((s_l[b * E + e] + 0.0) + (s_star[e] ? lamw : 0.0) - zmax);
        den = warp_sum(den);
    }
    double p = 0.0;
    int my_sel = 0;
    if (lane < k) {
        my_sel = s_sel[b * k + lane];
        const double zs = s_l[b * E + my_sel] + (s_star[my_sel] ? lamw : 0.0);
        p = exp_once(zs - zmax) / den;
    }
    if (sh.renorm) {
        const double tot = warp_sum(p);
        p /= tot;
    }
    if (lane < k) {
        s_pw[b * k + lane] = (float)p;
        sel_idx[b * k + lane] = my_sel;
        sel_w[b * k + lane] = (float)p;
        // the token's bit in the expert's 64-bit mask: a native 32-bit shared-memory atomic on the
        // half that holds it (a 64-bit atomicOr would be a compare-and-swap loop)
        atomicOr(reinterpret_cast<unsigned *>(&s_mask[my_sel]) + (b >> 5), 1u << (b & 31));
    }
}

// Gating of one batch by one thread block of at least two warps.
// s_l: shared memory for B*E doubles (the logits, copied from the workspace).
template <int JE>
__device__ __forceinline__ void gating_block(const Shape &sh, int B, const Workspace &ws, const float *__restrict__ conf,
                                             int has_gate, int32_t *__restrict__ sel_idx, float *__restrict__ sel_w,
                                             int32_t *__restrict__ n_unique, double *s_l)
{
    __shared__ unsigned long long s_gk[kMaxExperts];
    __shared__ unsigned char s_star[kMaxExperts];
    __shared__ double s_w[kMaxTokens], s_lam[kMaxTokens], s_zmax[kMaxTokens], s_den[kMaxTokens];
    __shared__ int s_sel[kMaxTokens * kMaxTopK];
    __shared__ float s_pw[kMaxTokens * kMaxTopK];
    __shared__ unsigned long long s_mask[kMaxExperts];
    __shared__ int s_cnt[kMaxExperts], s_off[kMaxExperts + 1], s_pos[kMaxExperts];
    __shared__ int s_U;

    const int tid = threadIdx.x, nt = blockDim.x, warp = tid >> 5, lane = tid & 31, nw = nt >> 5;
    const int E = sh.E, k = sh.k, cap = sh.cap;
    const bool bias_on = sh.alpha > 0.0 && cap < E && k < E;

#pragma unroll 1
    for (int i = tid; i < B * E; i += nt) s_l[i] = __ldcg(&ws.logits[i]);
#pragma unroll 1
    for (int b = tid; b < B; b += nt) s_w[b] = conf ? (double)conf[b] : 1.0;
#pragma unroll 1
    for (int e = tid; e < E; e += nt) { s_star[e] = 0; s_mask[e] = 0ull; }
    __syncthreads();

    // Two independent pieces run side by side on disjoint warps: the last cw warps pick the
    // reuse-reward set E* (Eq. 4 aggregation, TopCap), the others take the per-token order
    // statistics (lambda_b, softmax denominator).
    const int cw = bias_on ? max(1, min(nw / 2, nw - B)) : 0, tw = nw - cw;
    if (warp >= tw) {
        const int ct = tid - tw * 32, cn = cw * 32;
        // Eq. 4: g_e = sum_b w_b l_{b,e}, tokens in ascending order
#pragma unroll 1
        for (int e = ct; e < E; e += cn) {
            double g = 0.0;
#pragma unroll 1
            for (int b = 0; b < B; ++b) g = fma(s_w[b], s_l[b * E + e], g);
            s_gk[e] = dkey(g);
        }
        asm volatile("bar.sync 1, %0;" ::"r"(cn) : "memory");
        // TopCap by rank in the order (g descending, id ascending)
#pragma unroll 1
        for (int e = ct; e < E; e += cn) {
            const unsigned long long ge = s_gk[e];
            int rank = 0;
#pragma unroll 4
            for (int o = 0; o < E; ++o) {
                const unsigned long long go = s_gk[o];
                rank += (go > ge) | ((go == ge) & (o < e));
            }
            s_star[e] = rank < cap;
        }
    } else {
#pragma unroll 1
        for (int b = warp; b < B; b += tw) {
            gate_stats<JE>(sh, b, bias_on, s_l, s_lam, s_zmax, s_den, lane);
        }
    }
    __syncthreads();

#pragma unroll 1
    for (int b = warp; b < B; b += nw) {
        gate_select<JE>(sh, b, s_l, s_star, s_lam, s_zmax, s_den, s_sel, s_pw, s_mask, sel_idx, sel_w, lane);
    }
    __syncthreads();

    // union, unique count, exclusive scan, list of active experts: warp 0, lane owns a run of experts
    if (tid < 32) {
        const int C = (E + 31) >> 5, e0 = tid * C;
        int sum = 0, act = 0;
#pragma unroll 1
        for (int i = 0; i < C; ++i) {
            const int e = e0 + i;
            if (e < E) {
                const int c = __popcll(s_mask[e]);
                s_cnt[e] = c;
                sum += c;
                act += c > 0;
            }
        }
        int xs = sum, xa = act;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, xs, o), u = __shfl_up_sync(0xffffffffu, xa, o);
            if (tid >= o) { xs += t; xa += u; }
        }
        int off = xs - sum, pos = xa - act;
#pragma unroll 1
        for (int i = 0; i < C; ++i) {
            const int e = e0 + i;
            if (e < E) {
                s_off[e] = off;
                s_pos[e] = pos;
                off += s_cnt[e];
                pos += s_cnt[e] > 0;
            }
        }
        if (tid == 31) { s_off[E] = xs; s_U = xa; }
    }
    __syncthreads();
    const int U = s_U, n_routed = B * k;
#pragma unroll 1
    for (int e = tid; e < E; e += nt) {
        ws.counts[e] = s_cnt[e];
        ws.offsets[e] = s_off[e];
        if (s_cnt[e] > 0) {
            ws.active[s_pos[e]] = e;
            if (ws.gtab) {
                ws.gtab[2 * s_pos[e]] = make_uint4((unsigned)e, (unsigned)s_cnt[e], (unsigned)s_off[e], 0u);
                ws.gtab[2 * s_pos[e] + 1] = make_uint4((unsigned)s_mask[e], (unsigned)(s_mask[e] >> 32), 0u, 0u);
            }
        }
    }
    // bucket the (token, choice) pairs: tokens ascending inside an expert
#pragma unroll 1
    for (int i = tid; i < n_routed; i += nt) {
        const int b = i / k;
        const int e = s_sel[i];
        const int pos = s_off[e] + __popcll(s_mask[e] & ((1ull << b) - 1ull));
        ws.slot_token[pos] = b;
        ws.slot_w[pos] = s_pw[i];
    }
    // shared experts: every token, weight c_b
#pragma unroll 1
    for (int i = tid; i < sh.n_sh * B; i += nt) {
        const int s = i / B, b = i - s * B;
        float c = 1.0f;
        if (has_gate) c = (float)(1.0 / (1.0 + exp_once(-__ldcg(&ws.gate_logit[b]))));
        ws.slot_token[n_routed + i] = b;
        ws.slot_w[n_routed + i] = c;
        if (b == 0) {
            ws.counts[E + s] = B;
            ws.offsets[E + s] = n_routed + s * B;
            ws.active[U + s] = E + s;
            if (ws.gtab) {
                const unsigned long long all = B >= 64 ? ~0ull : ((1ull << B) - 1ull);
                ws.gtab[2 * (U + s)] = make_uint4((unsigned)(E + s), (unsigned)B, (unsigned)(n_routed + s * B), 0u);
                ws.gtab[2 * (U + s) + 1] = make_uint4((unsigned)all, (unsigned)(all >> 32), 0u, 0u);
            }
        }
    }
#pragma unroll 1
    for (int e = tid; e < E; e += nt) ws.tokmask[e] = s_mask[e];
#pragma unroll 1
    for (int s = tid; s < sh.n_sh; s += nt) ws.tokmask[E + s] = B >= 64 ? ~0ull : ((1ull << B) - 1ull);
    if (sh.plan == 2) {
        // stage tables of the streaming kernel: per active group, its first phase-1 stage
        // (4 gate + 4 up rows each) and first phase-2 stage (8 down rows x one K-slice)
        __syncthreads();
#pragma unroll 1
        for (int e = tid; e < E; e += nt)
            s_cnt[e] = s_cnt[e] > 0 ? st_nks(sh.f, s_cnt[e], sh.op_cap, sh.d) * (sh.d / 8) : 0;   // phase-2 stages
        __syncthreads();
#pragma unroll 1
        for (int e = tid; e < E; e += nt) {
            if (s_mask[e]) {
                int pre = 0;
#pragma unroll 1
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
#pragma unroll 1
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
constexpr int kRouteTok = 16;   // most tokens accumulated per pass

// Buffers that the layer's later kernels accumulate into and that must start at zero; the
// routing blocks clear them (16-byte units) so that no separate fill precedes the layer.
// two bf16 values -> two binary16 values (round to nearest; exact for magnitudes in [2^-14, 65504])
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t u)
{
    const __half2 h = __floats2half2_rn(bf16_lo(u), bf16_hi(u));
    return *reinterpret_cast<const uint32_t *>(&h);
}

struct ZeroList {
    void *ptr[3];
    unsigned long long n16[3];
    // int4 tensor-core path: a binary16 copy of the bf16 hidden states whose columns are permuted
    // inside every group of 8 (position p holds column [0,4,1,5,2,6,3,7][p]), the order in which
    // the dequantising warps of the FFN kernel get the nibbles of a 32-bit word for free
    const uint4 *perm_src;
    uint4 *perm_dst;
    unsigned long long perm_n16;
    // logit pass: the tokens of a batch are split into this many groups, each with its own set of
    // row blocks (0 and 1: every row block takes all tokens)
    int groups;
};

// One pass of a router row over NT tokens b0 .. b0 + NT - 1 (indices past B - 1 repeat token
// B - 1, so that every load is unconditional and issued before the first use).
template <int ACT, int RT, int NT>
__device__ __forceinline__ void route_pass(const Shape &sh, int B, int b0, const Workspace &ws, int row, const uint8_t *wrow,
                                           const void *__restrict__ hidden, double *s_part)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, d = sh.d;
    const size_t ab = ACT == DT_F32 ? 4 : 2;
    double acc[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t) acc[t] = 0.0;
    for (int c = tid * 4; c < d; c += kRouteThreads * 4) {
        float w[4], x[NT][4];
        load4_plain<RT>(wrow, c, w);
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const int bt = min(b0 + t, B - 1);
            load4_plain<ACT>(reinterpret_cast<const uint8_t *>(hidden) + (size_t)bt * d * ab, c, x[t]);
        }
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[t] = fma((double)w[i], (double)x[t][i], acc[t]);
    }
#pragma unroll
    for (int t = 0; t < NT; ++t) {
        const double s = warp_sum(acc[t]);
        if (lane == 0) s_part[warp * kRouteTok + t] = s;
    }
    __syncthreads();
    if (tid < NT && b0 + tid < B) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kRouteThreads / 32; ++w) s += s_part[w * kRouteTok + tid];
        if (row < sh.E) ws.logits[(size_t)(b0 + tid) * sh.E + row] = s;
        else ws.gate_logit[b0 + tid] = s;
    }
    __syncthreads();
}

// Router logits and gating in one launch.  A block computes one row of the router (row E is the
// shared-expert gate vector) against one group of the batch's tokens in float64; block 0 then
// runs the gating for the whole batch once every block has arrived (atomic ticket).
// Dynamic shared memory: max(B * E, 16 * kRouteTok) doubles.
// JE: experts per lane in the gating (2, 4 or 8 for up to 64, 128, 256 experts): a kernel of its own
// for each, so that the gating code of a launch is one straight piece
template <int ACT, int RT, int JE>
__global__ void __launch_bounds__(kRouteThreads)
route_kernel(Shape sh, int B, Workspace ws, const void *__restrict__ hidden, const void *__restrict__ router,
             const void *__restrict__ sh_scale, const float *__restrict__ conf, int32_t *__restrict__ sel_idx,
             float *__restrict__ sel_w, int32_t *__restrict__ n_unique, ZeroList zl)
{
    extern __shared__ double s_dyn[];
    __shared__ int s_last;
    const int tid = threadIdx.x;
    // Programmatic dependent launch: everything this kernel writes is read by the previous
    // layer's kernels, so it waits for them first; the FFN kernel that follows may come up now
    // and do its own set-up (both instructions do nothing in a plain launch).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#pragma unroll
    for (int z = 0; z < 3; ++z) {
        uint4 *p = reinterpret_cast<uint4 *>(zl.ptr[z]);
        for (unsigned long long i = (unsigned long long)blockIdx.x * kRouteThreads + tid; i < zl.n16[z];
             i += (unsigned long long)gridDim.x * kRouteThreads)
            p[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    for (unsigned long long i = (unsigned long long)blockIdx.x * kRouteThreads + tid; i < zl.perm_n16;
         i += (unsigned long long)gridDim.x * kRouteThreads) {
        const uint4 v = zl.perm_src[i];             // halves h0..h7 (bf16)
        zl.perm_dst[i] = make_uint4(bf16x2_to_f16x2(__byte_perm(v.x, v.z, 0x5410)), bf16x2_to_f16x2(__byte_perm(v.x, v.z, 0x7632)),
                                    bf16x2_to_f16x2(__byte_perm(v.y, v.w, 0x5410)), bf16x2_to_f16x2(__byte_perm(v.y, v.w, 0x7632)));
    }
    // blocks past the router's rows exist only to help with the clearing and the copy above (a
    // layer with few experts and wide accumulators would otherwise clear megabytes with a few blocks)
    // A row block takes one router row and one group of tokens: a larger batch is split over
    // several sets of row blocks (as many as fit on the SMs beside each other), because a block
    // takes 16 tokens per pass and its passes run one after the other (B = 64: 22 us in one set).
    const int n_rows = sh.E + (sh_scale ? 1 : 0);
    const int n_grp = zl.groups > 1 ? zl.groups : 1, n_arrive = n_rows * n_grp;
    if ((int)blockIdx.x >= n_arrive) return;
    const int row = (int)blockIdx.x % n_rows, grp = (int)blockIdx.x / n_rows, d = sh.d;
    const int tg = 4 * ((B + 4 * n_grp - 1) / (4 * n_grp));            // tokens per group, a multiple of 4
    const int b_lo = min(B, grp * tg), b_hi = min(B, b_lo + tg);
    const size_t rb = RT == DT_F32 ? 4 : 2;
    const uint8_t *wrow = row < sh.E ? reinterpret_cast<const uint8_t *>(router) + (size_t)row * d * rb
                                     : reinterpret_cast<const uint8_t *>(sh_scale);
    for (int b0 = b_lo; b0 < b_hi;) {
        const int left = b_hi - b0;
        if (left > 8) { route_pass<ACT, RT, 16>(sh, B, b0, ws, row, wrow, hidden, s_dyn); b0 += 16; }
        else if (left > 4) { route_pass<ACT, RT, 8>(sh, B, b0, ws, row, wrow, hidden, s_dyn); b0 += 8; }
        else { route_pass<ACT, RT, 4>(sh, B, b0, ws, row, wrow, hidden, s_dyn); b0 += 4; }
    }
    // Block 0 runs the gating once every row has arrived (its SM tends to be the same from layer
    // to layer, so part of the gating code is still in its instruction cache: measured 0.6 % of
    // a layer against letting the last block to arrive do it).  Every block takes a ticket with
    // release and acquire semantics by one thread.  The block that takes the last ticket puts the
    // counter back to zero (nobody else touches it before the next launch) and publishes, in the
    // word behind the counter, the token that block 0 wrote two words further in front of its own ticket;
    // block 0 polls, bounded, for exactly that token.  So a wait that ran out leaves nothing
    // behind: the late blocks still reset the counter, and what they publish afterwards is the
    // token of a launch that is over, which no later launch waits for.  The barriers on both
    // sides extend the ordering to the block's other threads; the other blocks wait for nothing.
    if (tid == 0) {
        unsigned token = 0u;
        if (blockIdx.x == 0) {
            // differs from launch to launch (a wrapped nanosecond timer; never 0)
            unsigned long long gt;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt));
            token = (unsigned)gt | 1u;
            asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(ws.ticket + 2), "r"(token) : "memory");
        }
        unsigned t;
        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(t) : "l"(ws.ticket) : "memory");
        const bool last = t == (unsigned)n_arrive - 1;
        if (last) {
            unsigned tk;
            asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(tk) : "l"(ws.ticket + 2) : "memory");
            asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(ws.ticket), "r"(0u) : "memory");
            if (blockIdx.x != 0)
                asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(ws.ticket + 1), "r"(tk) : "memory");
        }
        int ok = (blockIdx.x == 0 && last) ? 1 : 0;
        if (blockIdx.x == 0 && !last) {
            for (unsigned i = 0; i < (1u << 22); ++i) {
                unsigned v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ws.ticket + 1) : "memory");
                if (v == token) { ok = 1; break; }
                __nanosleep(20);
            }
            if (!ok) atomicExch(ws.status, ST_TICKET_TIMEOUT);
        }
        s_last = ok;
    }
    __syncthreads();
    if (!s_last) return;
    gating_block<JE>(sh, B, ws, conf, sh_scale ? 1 : 0, sel_idx, sel_w, n_unique, s_dyn);
}

}  // namespace s2moe
