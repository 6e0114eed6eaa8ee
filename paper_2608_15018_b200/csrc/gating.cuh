// Reuse-aware expert gating (Sec. 4.2) of one draft batch on given float64 router logits,
// written for a GROUP of warps of a thread block (the whole block of the routing kernel, or the
// warps of the fused layer kernel that have nothing else to do while the layer starts):
//
//   Eq. 4 aggregation g_e = sum_b w_b l_{b,e}, TopCap (E* = the cap experts of largest g),
//   lambda_b = alpha (l_(1) - l_(k+1)), biased top-k in the order (l' descending, l descending,
//   id ascending), mixing weights, union / unique count.
//
// Everything that decides an index is an exact comparison of float64 values through
// order-preserving 64-bit integer keys.  One warp per token; a selection is k rounds of a
// warp-wide maximum.  (Measured against it on the same GPU: sorting every token's experts with a
// bitonic network and merging the two lists that the bias leaves in order is data-independent
// and has no long chain, but needs about three times the instructions per token, and with several
// tokens' warps on one scheduler that made the gating 1 us slower at 8 tokens.)
#pragma once

#include "common.cuh"

namespace s2moe {

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One copy of the double-precision exponential for the whole gating: the gating runs once per
// layer, so its cost follows the amount of distinct code.
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

// a group of warps of one block and the two named barriers that belong to it
struct GateGroup {
    int t, n, bar;      // thread index inside the group, threads of the group (a multiple of 32, at least 64),
                        // first of two consecutive hardware barriers
};
__device__ __forceinline__ void gate_sync(const GateGroup &g)
{
    asm volatile("bar.sync %0, %1;" ::"r"(g.bar), "r"(g.n) : "memory");
}

// shared memory of the gating; the results stay here for whoever called it
struct GateMem {
    unsigned long long *mask;   // [E] bit b: token b selected the expert
    unsigned long long *gk;     // [E] keys of the aggregated importance g_e
    double *lam, *zmax, *den;   // [B] lambda_b, softmax maximum and denominator of the original logits
    int *sel;                   // [B * k] selected experts in selection order
    float *pw;                  // [B * k] their mixing weights
    int *cnt, *off, *pos;       // [E] tokens per expert, [E + 1] first slot, [E] index in the active list
    int *U;                     // [1] distinct selected experts
    unsigned *star32;           // [8] E* as bit words (bit i of word j: expert i + 32 j)
    unsigned *topk;             // [B][J] every token's first k experts by original logit, same bit layout (bias on only)
    unsigned char *star;        // [E] member of E*
};
__host__ __device__ __forceinline__ size_t gate_mem_bytes(int E, int B, int k)
{
    return 16 * (size_t)E + 24 * (size_t)B + 8 * (size_t)B * k + 4 * (size_t)(3 * E + 1) + 4 + 32 + 4 * (size_t)B * 8 +
           (((size_t)E + 15) & ~(size_t)15) + 16;
}
__device__ __forceinline__ GateMem gate_mem_carve(void *base, int E, int B, int k)
{
    GateMem m;
    uint8_t *p = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(base) + 7) & ~(uintptr_t)7);
    m.mask = reinterpret_cast<unsigned long long *>(p); p += 8 * (size_t)E;
    m.gk = reinterpret_cast<unsigned long long *>(p); p += 8 * (size_t)E;
    m.lam = reinterpret_cast<double *>(p); p += 8 * (size_t)B;
    m.zmax = reinterpret_cast<double *>(p); p += 8 * (size_t)B;
    m.den = reinterpret_cast<double *>(p); p += 8 * (size_t)B;
    m.sel = reinterpret_cast<int *>(p); p += 4 * (size_t)B * k;
    m.pw = reinterpret_cast<float *>(p); p += 4 * (size_t)B * k;
    m.cnt = reinterpret_cast<int *>(p); p += 4 * (size_t)E;
    m.off = reinterpret_cast<int *>(p); p += 4 * (size_t)(E + 1);
    m.pos = reinterpret_cast<int *>(p); p += 4 * (size_t)E;
    m.U = reinterpret_cast<int *>(p); p += 4;
    m.star32 = reinterpret_cast<unsigned *>(p); p += 32;
    m.topk = reinterpret_cast<unsigned *>(p); p += 4 * (size_t)B * 8;
    m.star = p;
    return m;
}

// Order statistics of one token's original logits, one warp per token (lane owns experts lane,
// lane + 32, ...): lambda_b = alpha (l_(1) - l_(k+1)) by k + 1 rounds of a warp-wide maximum over
// integer keys, winners in the exact order (logit descending, id ascending); the token's first k
// experts in that order as bit words (word j, bit i: expert i + 32 j; s_topk, or NULL); and, for
// weight_mode 0 and unless the caller leaves it to gate_select (with_den false), the softmax
// denominator over the original logits.
// TRACK: the membership words are wanted (only then do equal logits have to be told apart: the
// order statistics themselves are the same whichever of two equal logits wins a round).
template <int J, bool TRACK>
__device__ __forceinline__ void gate_stats(const Shape &sh, int b, bool bias_on, const double *s_l, double *s_lam,
                                           double *s_zmax, double *s_den, unsigned *s_topk, bool with_den, int lane)
{
    const unsigned full = 0xffffffffu;
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
    unsigned won = 0;                                    // bit j: element j of this lane is among the first k
    if constexpr (J == 2) {
        // two elements per lane: the lane offers its first one in the order and, once that has won a
        // round, the other (a key of 0 = nothing left); a round is one reduction and one ballot
        const bool first0 = k1[0] >= k1[1];
        unsigned long long cur = first0 ? k1[0] : k1[1], nxt = first0 ? k1[1] : k1[0];
        unsigned cj = first0 ? 0u : 1u;
#pragma unroll 1
        for (int r = 0; r < rounds; ++r) {
            unsigned hb = warp_max_holders(cur, cur != 0ull);
            if (TRACK && __popc(hb) > 1) {               // equal logits: lower expert id first
                const bool hold = (hb >> lane) & 1u;
                const unsigned me = __reduce_min_sync(full, hold ? (unsigned)lane + 32u * cj : 0xffffffffu);
                hb = __ballot_sync(full, hold && (unsigned)lane + 32u * cj == me);
            }
            const int wl = __ffs(hb) - 1;
            if (r == 0) top1 = shfl_key(cur, wl);
            if (r == k) kth = shfl_key(cur, wl);
            if (lane == wl) {                            // drop the winner
                if (TRACK) { if (r < k) won |= 1u << cj; cj ^= 1u; }
                cur = nxt; nxt = 0ull;
            }
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
            unsigned hb = warp_max_holders(lm, alive != 0u);
            if (TRACK && __popc(hb) > 1) {               // equal logits: lower expert id first
                const bool hold = (hb >> lane) & 1u;
                const unsigned me = __reduce_min_sync(full, hold ? (unsigned)(lane + 32 * bj) : 0xffffffffu);
                hb = __ballot_sync(full, hold && (unsigned)(lane + 32 * bj) == me);
            }
            const int wl = __ffs(hb) - 1;
            if (r == 0) top1 = shfl_key(lm, wl);
            if (r == k) kth = shfl_key(lm, wl);
            if (lane == wl) {                            // drop the winner
                if (TRACK && r < k) won |= 1u << bj;
                alive &= ~(1u << bj);
            }
        }
    }
    if (TRACK && s_topk) {
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const unsigned word = __ballot_sync(full, (won >> j) & 1u);
            if (lane == 0) s_topk[b * J + j] = word;
        }
    }
    const double ztop = dkey_value(top1);
    double den = 0.0;
    if (!sh.weight_mode && with_den) {
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
                                            float *__restrict__ sel_w, bool have_den, int lane)
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
    if (!sh.weight_mode && !have_den) {
        den = 0.0;
#pragma unroll 1
        for (int e = lane; e < E; e += 32) den += exp_once((s_l[b * E + e] + 0.0) - zmax);
        den = warp_sum(den);
    }
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
        if (sel_idx) {
            sel_idx[b * k + lane] = my_sel;
            sel_w[b * k + lane] = (float)p;
        }
        // the token's bit in the expert's 64-bit mask: a native 32-bit shared-memory atomic on the
        // half that holds it (a 64-bit atomicOr would be a compare-and-swap loop)
        atomicOr(reinterpret_cast<unsigned *>(&s_mask[my_sel]) + (b >> 5), 1u << (b & 31));
    }
}

// Steps O2..O5 for B tokens on `s_l` [B][E] (logits) and `s_w` [B] (confidences), both in SHARED
// memory and visible to the group (every row is read several times and E* needs all of them, so a
// caller stages them once: one memory round trip for the whole gating), by the warps of `gg`, in
// two parts.  After gating_part1 (the group is synchronised) gm holds E* (star, star32), lambda_b and
// every token's first k experts by original logit (topk: with the bias on these are the experts
// that the token keeps whenever they are in E*, see the fused kernel); after gating_part2 sel / pw
// in selection order, the per-expert token masks and counts, the exclusive scan `off`, the index
// `pos` of every active expert in the ascending list of active experts, and U.  sel_idx / sel_w
// (global, or NULL) receive the selection and the weights.  den_early: the softmax denominators are
// taken in part 1 (beside the search for E*), else in part 2.
// J: experts per lane (2, 4, 8 for up to 64, 128, 256 experts).
// E* by cn threads (thread ct of them; a multiple of 32) that meet on hardware barrier `bar`:
// Eq. 4 aggregation, TopCap by rank.  gm.star and gm.star32 must have been cleared.
__device__ __forceinline__ void gating_estar(const Shape &sh, int B, const double *__restrict__ s_l,
                                             const double *__restrict__ s_w, const GateMem &gm, int ct, int cn, int bar)
{
    const int E = sh.E, cap = sh.cap;
    // Eq. 4: g_e = sum_b w_b l_{b,e}, tokens in ascending order
#pragma unroll 1
    for (int e = ct; e < E; e += cn) {
        double g = 0.0;
#pragma unroll 1
        for (int b = 0; b < B; ++b) g = fma(s_w[b], s_l[b * E + e], g);
        gm.gk[e] = dkey(g);
    }
    asm volatile("bar.sync %0, %1;" ::"r"(bar), "r"(cn) : "memory");
    // TopCap by rank in the order (g descending, id ascending)
#pragma unroll 1
    for (int e = ct; e < E; e += cn) {
        const unsigned long long ge = gm.gk[e];
        int rank = 0;
#pragma unroll 4
        for (int o = 0; o < E; ++o) {
            const unsigned long long go = gm.gk[o];
            rank += (go > ge) | ((go == ge) & (o < e));
        }
        gm.star[e] = rank < cap;
        if (rank < cap) atomicOr(&gm.star32[e >> 5], 1u << (e & 31));
    }
}

template <int J>
__device__ __forceinline__ void gating_part1(const Shape &sh, int B, const double *__restrict__ s_l,
                                             const double *__restrict__ s_w, const GateGroup gg, const GateMem gm, bool den_early,
                                             bool star_done = false, bool want_topk = false)
{
    const int tid = gg.t, nt = gg.n, warp = tid >> 5, lane = tid & 31, nw = nt >> 5;
    const int E = sh.E, k = sh.k, cap = sh.cap;
    const bool bias_on = sh.alpha > 0.0 && cap < E && k < E;
#pragma unroll 1
    for (int e = tid; e < E; e += nt) {
        if (!star_done) gm.star[e] = 0;
        gm.mask[e] = 0ull;
    }
    if (tid < 8 && !star_done) gm.star32[tid] = 0u;
    gate_sync(gg);

    // E* on the last cw warps (unless the caller has it already), the per-token order statistics
    // (lambda_b, softmax denominator) on the others, side by side: half of the warps when the batch
    // leaves that many idle, else as many as it leaves, at least one (measured against letting the
    // first warps find E* and then take tokens with everybody: 1.3 us slower at 16 tokens).
    const int cw = (!bias_on || star_done) ? 0 : max(1, min(nw / 2, nw - B));
    const bool side = cw > 0;
    const int c0 = nw - cw;                            // first of the cw warps
    if (warp >= c0 && warp < c0 + cw) gating_estar(sh, B, s_l, s_w, gm, tid - c0 * 32, cw * 32, gg.bar + 1);
    if (!side || warp < c0) {
        const int tw = side ? c0 : nw;
        if (bias_on && want_topk) {
#pragma unroll 1
            for (int b = warp; b < B; b += tw)
                gate_stats<J, true>(sh, b, bias_on, s_l, gm.lam, gm.zmax, gm.den, gm.topk, den_early, lane);
        } else {
#pragma unroll 1
            for (int b = warp; b < B; b += tw)
                gate_stats<J, false>(sh, b, bias_on, s_l, gm.lam, gm.zmax, gm.den, nullptr, den_early, lane);
        }
    }
    gate_sync(gg);
}

// The expert with the largest original logit of token b (equal logits: the lower id), by one warp.
template <int J>
__device__ __forceinline__ int gate_top1(const Shape &sh, int b, const double *s_l, int lane)
{
    const unsigned full = 0xffffffffu;
    unsigned long long best = 0ull;
    int be = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < J; ++j) {
        const int e = lane + 32 * j;
        if (e < sh.E) {
            const unsigned long long kk = dkey(s_l[b * sh.E + e]);
            if (kk > best) { best = kk; be = e; }          // (e ascends with j: the first of equal keys stays)
        }
    }
    const unsigned hb = warp_max_holders(best, be != 0x7fffffff);
    return (int)__reduce_min_sync(full, ((hb >> lane) & 1u) ? (unsigned)be : 0xffffffffu);
}

// early32 (or NULL): bit words of experts that go to the front of the active list and of the slot
// order, ascending among themselves (every one of them must have been selected by some token); the
// other active experts follow in ascending order.
template <int J>
__device__ __forceinline__ void gating_part2(const Shape &sh, int B, const double *__restrict__ s_l, const GateGroup gg,
                                             const GateMem gm, int32_t *__restrict__ sel_idx, float *__restrict__ sel_w,
                                             bool den_early, const unsigned *early32 = nullptr)
{
    const int tid = gg.t, nt = gg.n, warp = tid >> 5, lane = tid & 31, nw = nt >> 5;
    const int E = sh.E;
#pragma unroll 1
    for (int b = warp; b < B; b += nw)
        gate_select<J>(sh, b, s_l, gm.star, gm.lam, gm.zmax, gm.den, gm.sel, gm.pw, gm.mask, sel_idx, sel_w, den_early, lane);
    gate_sync(gg);

    // union, unique count, exclusive scan, list of active experts: warp 0, lane owns a run of experts
    if (tid < 32) {
        const int C = (E + 31) >> 5, e0 = lane * C;
        int sum = 0, act = 0, esum = 0, eact = 0;        // all experts of the run; the early ones among them
#pragma unroll 1
        for (int i = 0; i < C; ++i) {
            const int e = e0 + i;
            if (e < E) {
                const int c = __popcll(gm.mask[e]);
                gm.cnt[e] = c;
                sum += c;
                act += c > 0;
                if (early32 && ((early32[e >> 5] >> (e & 31)) & 1u)) { esum += c; eact += c > 0; }
            }
        }
        int xs = sum, xa = act, ys = esum, ya = eact;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, xs, o), u = __shfl_up_sync(0xffffffffu, xa, o);
            if (lane >= o) { xs += t; xa += u; }
            if (early32) {
                const int t2 = __shfl_up_sync(0xffffffffu, ys, o), u2 = __shfl_up_sync(0xffffffffu, ya, o);
                if (lane >= o) { ys += t2; ya += u2; }
            }
        }
        // slots and list positions: the early experts first, then the rest
        const int te = early32 ? __shfl_sync(0xffffffffu, ys, 31) : 0, ne = early32 ? __shfl_sync(0xffffffffu, ya, 31) : 0;
        int eoff = ys - esum, epos = ya - eact;
        int off = te + (xs - sum) - eoff, pos = ne + (xa - act) - epos;
#pragma unroll 1
        for (int i = 0; i < C; ++i) {
            const int e = e0 + i;
            if (e < E) {
                const int c = gm.cnt[e];
                if (early32 && ((early32[e >> 5] >> (e & 31)) & 1u)) {
                    gm.off[e] = eoff; gm.pos[e] = epos;
                    eoff += c; epos += c > 0;
                } else {
                    gm.off[e] = off; gm.pos[e] = pos;
                    off += c; pos += c > 0;
                }
            }
        }
        if (lane == 31) { gm.off[E] = xs; *gm.U = xa; }
    }
    gate_sync(gg);
}

}  // namespace s2moe
