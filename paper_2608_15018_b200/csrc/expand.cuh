// Routing-aware adaptive speculative expansion (Sec. 4.1): predicted expert sets as bit
// masks, marginal verification cost (Eq. 2), utility (Eq. 3) and the greedy admission loop.
// The step that chooses the draft batch which the verification layer then runs on.
#pragma once

#include <cstdint>

namespace s2moe {

constexpr int kExpandMaxCand = 256;     // candidates per call (one thread each)
constexpr int kExpandMaxWords = 512;    // n_layers * ceil(n_experts / 64)

// masks[t * stride + w]: bit (e % 64) of word (e / 64) set for every expert e in sel_idx[t][*]
__global__ void expert_masks_kernel(const int32_t *__restrict__ sel_idx, int n_tokens, int k, int words,
                                    unsigned long long *__restrict__ masks, int stride)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_tokens) return;
    for (int w = 0; w < words; ++w) {
        unsigned long long m = 0ull;
        for (int j = 0; j < k; ++j) {
            const int e = sel_idx[t * k + j];
            if ((e >> 6) == w) m |= 1ull << (e & 63);
        }
        masks[(size_t)t * stride + w] = m;
    }
}

// One block; thread i owns candidate i.  All arithmetic that decides an admission is float64
// with every operation rounded on its own (no fused multiply-add), so that the decisions are
// those of the plain definition.
__global__ void __launch_bounds__(kExpandMaxCand)
adaptive_expand_kernel(int n, int lw, const int32_t *__restrict__ parent, const float *__restrict__ p_tok,
                       const unsigned long long *__restrict__ masks, const float *__restrict__ c_draft, float t_ar,
                       float t_exp, int32_t *__restrict__ admitted, int32_t *__restrict__ order,
                       int32_t *__restrict__ n_admitted, unsigned long long *__restrict__ union_out)
{
    __shared__ double s_p[kExpandMaxCand];
    __shared__ int s_adm[kExpandMaxCand];
    __shared__ unsigned long long s_union[kExpandMaxWords];
    __shared__ double s_wu[kExpandMaxCand / 32];
    __shared__ int s_wi[kExpandMaxCand / 32];
    __shared__ int s_best, s_count, s_bad;

    const int i = threadIdx.x, lane = i & 31, warp = i >> 5, nw = blockDim.x >> 5;
    if (i < n) s_adm[i] = 0;
    for (int w = i; w < lw; w += blockDim.x) s_union[w] = 0ull;
    if (i == 0) {
        // prefix confidence p_i = p_parent * p_{i,j}; parents precede their children.  A parent
        // index that does not (>= the candidate's own) is not followed: the candidate gets
        // confidence 0, is never eligible (nor are its descendants) and the call reports it
        int bad = 0;
        for (int c = 0; c < n; ++c) {
            const int a = parent[c];
            if (a >= c) { s_p[c] = 0.0; bad = 1; continue; }
            s_p[c] = a < 0 ? (double)p_tok[c] : __dmul_rn(s_p[a], (double)p_tok[c]);
        }
        s_count = 0;
        s_bad = bad;
    }
    __syncthreads();
    const int par_in = i < n ? parent[i] : -1;
    const bool malformed = i < n && par_in >= i;
    const int par = malformed ? -1 : par_in;
    const double cd = (i < n && c_draft) ? (double)c_draft[i] : 0.0;
    const double benefit = i < n ? __dmul_rn(s_p[i], (double)t_ar) : 0.0;
    const double neg_inf = -__longlong_as_double(0x7ff0000000000000ll), pos_inf = -neg_inf;

    for (int step = 0; step < n; ++step) {
        double u = neg_inf;
        if (i < n && !malformed && !s_adm[i] && (par < 0 || s_adm[par])) {
            int fresh = 0;                                         // Eq. 2: | E_i \ union |, all layers
            for (int w = 0; w < lw; ++w) fresh += __popcll(masks[(size_t)i * lw + w] & ~s_union[w]);
            const double cost = __dadd_rn(__dmul_rn((double)fresh, (double)t_exp), cd);
            u = cost == 0.0 ? pos_inf : __ddiv_rn(benefit, cost);  // Eq. 3
        }
        // largest utility, lowest index on ties
        int bi = i;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const double ou = __shfl_down_sync(0xffffffffu, u, o);
            const int oi = __shfl_down_sync(0xffffffffu, bi, o);
            if (ou > u || (ou == u && oi < bi)) { u = ou; bi = oi; }
        }
        if (lane == 0) { s_wu[warp] = u; s_wi[warp] = bi; }
        __syncthreads();
        if (i == 0) {
            double bu = s_wu[0];
            int b = s_wi[0];
            for (int w = 1; w < nw; ++w)
                if (s_wu[w] > bu || (s_wu[w] == bu && s_wi[w] < b)) { bu = s_wu[w]; b = s_wi[w]; }
            if (bu >= 1.0) {
                s_adm[b] = 1;
                order[s_count++] = b;
                s_best = b;
            } else {
                s_best = -1;
            }
        }
        __syncthreads();
        const int b = s_best;
        if (b < 0) break;
        for (int w = i; w < lw; w += blockDim.x) s_union[w] |= masks[(size_t)b * lw + w];
        __syncthreads();
    }
    __syncthreads();
    if (i < n) {
        admitted[i] = s_adm[i];
        if (i >= s_count) order[i] = -1;
    }
    if (i == 0) *n_admitted = s_bad ? -1 : s_count;      // -1: parent[] was malformed
    if (union_out)
        for (int w = i; w < lw; w += blockDim.x) union_out[w] = s_union[w];
}

}  // namespace s2moe
