// Router logits and reuse-aware expert gating (Sec. 4.2) for one draft batch.
//
//   route_kernel : l_{b,e} = h_b . W_r[e] (and the shared-expert gate logit) in float64, so
//                  that the discrete choices below do not depend on the summation order;
//                  block 0 then runs gating_block once every row has arrived:
//   gating_block : Eq. 4 aggregation, TopCap, lambda_b, biased top-k, mixing weights,
//                  union / unique count (gating.cuh), token->expert bucketing, stage tables.
#pragma once

#include "common.cuh"
#include "ffn_stream.cuh"
#include "gating.cuh"

namespace s2moe {


// What the expert kernels read of a finished gating (see gating_group for gm): the bucketing
// arrays in the workspace, tokens ascending inside an expert, the shared experts' groups behind
// the routed ones, and the stage tables of the streaming kernel.
__device__ __forceinline__ void gating_writeout(const Shape &sh, int B, const Workspace &ws, const GateMem &gm, int has_gate,
                                                int32_t *__restrict__ n_unique, const GateGroup gg)
{
    const int tid = gg.t, nt = gg.n;
    const int E = sh.E, k = sh.k;
    const int U = *gm.U, n_routed = B * k;
#pragma unroll 1
    for (int e = tid; e < E; e += nt) {
        ws.counts[e] = gm.cnt[e];
        ws.offsets[e] = gm.off[e];
        ws.tokmask[e] = gm.mask[e];
        if (gm.cnt[e] > 0) {
            ws.active[gm.pos[e]] = e;
            if (ws.gtab) {
                ws.gtab[2 * gm.pos[e]] = make_uint4((unsigned)e, (unsigned)gm.cnt[e], (unsigned)gm.off[e], 0u);
                ws.gtab[2 * gm.pos[e] + 1] = make_uint4((unsigned)gm.mask[e], (unsigned)(gm.mask[e] >> 32), 0u, 0u);
            }
        }
    }
    // bucket the (token, choice) pairs: tokens ascending inside an expert
#pragma unroll 1
    for (int i = tid; i < n_routed; i += nt) {
        const int b = i / k;
        const int e = gm.sel[i];
        const int pos = gm.off[e] + __popcll(gm.mask[e] & ((1ull << b) - 1ull));
        ws.slot_token[pos] = b;
        ws.slot_w[pos] = gm.pw[i];
    }
    // shared experts: every token, weight c_b
    const unsigned long long all = B >= 64 ? ~0ull : ((1ull << B) - 1ull);
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
            ws.tokmask[E + s] = all;
            if (ws.gtab) {
                ws.gtab[2 * (U + s)] = make_uint4((unsigned)(E + s), (unsigned)B, (unsigned)(n_routed + s * B), 0u);
                ws.gtab[2 * (U + s) + 1] = make_uint4((unsigned)all, (unsigned)(all >> 32), 0u, 0u);
            }
        }
    }
    if (sh.plan == 2) {
        // stage tables of the streaming kernel: per active group, its first phase-1 stage
        // (4 gate + 4 up rows each) and first phase-2 stage (8 down rows x one K-slice)
        gate_sync(gg);
#pragma unroll 1
        for (int e = tid; e < E; e += nt)
            gm.cnt[e] = gm.cnt[e] > 0 ? st_nks(sh.f, gm.cnt[e], sh.op_cap, sh.d) * (sh.d / 8) : 0;   // phase-2 stages
        gate_sync(gg);
#pragma unroll 1
        for (int e = tid; e < E; e += nt) {
            if (gm.mask[e]) {
                int pre = 0;
#pragma unroll 1
                for (int o = 0; o < e; ++o) pre += gm.cnt[o];
                const int a = gm.pos[e];
                ws.upfx1[a] = a * (sh.f / 4);
                ws.upfx2[a] = pre;
                ws.sync[a] = 0;
                if (a == U - 1) gm.off[0] = pre + gm.cnt[e];   // all routed phase-2 stages
            }
        }
        gate_sync(gg);
        if (tid == 0) {
            int t1 = U * (sh.f / 4), t2 = gm.off[0];
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

// Gating of one batch by a whole thread block (kRouteThreads threads) on the logits in the workspace.
// s_l: shared memory for B * E + B doubles (the logits and the confidences are staged there).
template <int JE>
__device__ __forceinline__ void gating_block(const Shape &sh, int B, const Workspace &ws, const float *__restrict__ conf,
                                             int has_gate, int32_t *__restrict__ sel_idx, float *__restrict__ sel_w,
                                             int32_t *__restrict__ n_unique, double *s_l, int ksplit, const double *__restrict__ lpart,
                                             int early = 0)
{
    __shared__ unsigned long long s_mask[kMaxExperts], s_gk[kMaxExperts];
    __shared__ unsigned s_early32[8];
    __shared__ double s_lam[kMaxTokens], s_zmax[kMaxTokens], s_den[kMaxTokens];
    __shared__ int s_sel[kMaxTokens * kMaxTopK];
    __shared__ float s_pw[kMaxTokens * kMaxTopK];
    __shared__ int s_cnt[kMaxExperts], s_off[kMaxExperts + 1], s_pos[kMaxExperts];
    __shared__ int s_U;
    __shared__ unsigned s_star32[8];
    __shared__ unsigned char s_star[kMaxExperts];
    GateMem gm;
    gm.mask = s_mask; gm.gk = s_gk; gm.lam = s_lam; gm.zmax = s_zmax; gm.den = s_den; gm.sel = s_sel; gm.pw = s_pw;
    gm.cnt = s_cnt; gm.off = s_off; gm.pos = s_pos; gm.U = &s_U; gm.star = s_star; gm.star32 = s_star32;
    gm.topk = reinterpret_cast<unsigned *>(s_sel);      // (the selection overwrites it: nobody reads it here)
    const GateGroup gg{(int)threadIdx.x, (int)blockDim.x, 0};
    double *s_w = s_l + B * sh.E;
    if (ksplit > 0) {
        // the pieces of a row added in ascending order (all loads first); the sums go back to the
        // workspace, where the write-out (gate logits) and debug reads find them
        const int n_rows = sh.E + has_gate;
#pragma unroll 1
        for (int i = gg.t; i < B * n_rows; i += gg.n) {
            const int b = i / n_rows, r = i - b * n_rows;
            double v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = q < ksplit ? __ldcg(&lpart[((size_t)q * B + b) * n_rows + r]) : 0.0;
            double acc = v[0];
#pragma unroll
            for (int q = 1; q < 8; ++q) acc += v[q];
            if (r < sh.E) { s_l[b * sh.E + r] = acc; ws.logits[b * sh.E + r] = acc; }
            else ws.gate_logit[b] = acc;
        }
    } else {
#pragma unroll 1
        for (int i = gg.t; i < B * sh.E; i += gg.n) s_l[i] = __ldcg(&ws.logits[i]);
    }
#pragma unroll 1
    for (int b = gg.t; b < B; b += gg.n) s_w[b] = conf ? (double)conf[b] : 1.0;
    if (early) {
        // The expert kernel is already resident (programmatic launch) and waits for this list: the
        // experts whose first projection it may stream while the gating below still runs.  A token's
        // first expert by original logit stays selected whatever E* turns out to be (the bias lifts
        // an expert by at most alpha (l_(1) - l_(k+1)) <= l_(1) - l_(k+1), so only the other k - 1 of
        // its first k can pass it), which the caller has checked for this layer's alpha (early == 2).
        // These experts lead the active list and the slot order, ascending, so that the expert
        // kernel knows their groups before it knows the others.
        if (gg.t < 8) s_early32[gg.t] = 0u;
        __syncthreads();                                  // the logits are staged, the words cleared
        if (early == 2) {
#pragma unroll 1
            for (int b = gg.t >> 5; b < B; b += gg.n >> 5) {
                const int e = gate_top1<JE>(sh, b, s_l, gg.t & 31);
                if ((gg.t & 31) == 0) atomicOr(&s_early32[e >> 5], 1u << (e & 31));
            }
        }
        __syncthreads();
        // one 64-bit word per 32 experts: the bits of the early experts under a tag of 1 (the words
        // were cleared before this grid let the expert kernel be scheduled), each released by itself,
        // so that whoever polls a word has its part of the list with the same load
        if (gg.t < ((sh.E + 31) >> 5)) {
            const unsigned long long v = (1ull << 32) | (unsigned long long)s_early32[gg.t];
            asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(reinterpret_cast<unsigned long long *>(ws.early) + gg.t), "l"(v)
                         : "memory");
        }
    }
    // (gating_group's first barrier orders these writes before the first read)
    gating_part1<JE>(sh, B, s_l, s_w, gg, gm, true);
    gating_part2<JE>(sh, B, s_l, gg, gm, sel_idx, sel_w, true, early ? s_early32 : nullptr);
    gating_writeout(sh, B, ws, gm, has_gate, n_unique, gg);
}

constexpr int kRouteThreads = 512;
constexpr int kRouteThreadsBig = 1024;
constexpr int kRouteTok = 16;   // most tokens accumulated per pass

// Buffers that the layer's later kernels accumulate into and that must start at zero; the
// routing blocks clear them (16-byte units) so that no separate fill precedes the layer.
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
    // logit pass by warp tasks (larger batches): ksplit > 0 pieces of the contraction per router row,
    // partial sums in lpart [piece][token][row] (see route_logit_tasks); 0: by row blocks
    int ksplit;
    double *lpart;
    // 1: the expert kernel behind this launch starts before the gating has ended (see gating_block);
    // 2: the same, and every token's first expert by original logit is known to stay selected
    int early;
};

// Router logits by the warps of the whole grid: a task is one router row (row E: the shared
// experts' gate vector) x 8 tokens x one piece of the contraction, float64 accumulation; its
// partial sums go to lpart[piece][token][row], which the gating adds up in a fixed order.
template <int ACT, int RT>
__device__ __forceinline__ void route_logit_tasks(const Shape &sh, int B, const void *__restrict__ hidden,
                                                  const void *__restrict__ router, const void *__restrict__ sh_scale,
                                                  double *__restrict__ lpart, int ksplit, int gwarp, int n_gwarps, int lane)
{
    const int d = sh.d, n_rows = sh.E + (sh_scale ? 1 : 0), n_tg = (B + 7) >> 3;
    const int len = ((d + 4 * ksplit - 1) / (4 * ksplit)) * 4;              // columns of a piece, a multiple of 4
    const int n_tasks = n_rows * n_tg * ksplit;
    const size_t rb = RT == DT_F32 ? 4 : 2, ab = ACT == DT_F32 ? 4 : 2;
#pragma unroll 1
    for (int task = gwarp; task < n_tasks; task += n_gwarps) {
        const int row = task % n_rows, rest = task / n_rows, tg = rest % n_tg, piece = rest / n_tg;
        const int c0 = piece * len, c1 = min(d, c0 + len), b0 = tg * 8;
        const uint8_t *wrow = row < sh.E ? reinterpret_cast<const uint8_t *>(router) + (size_t)row * d * rb
                                         : reinterpret_cast<const uint8_t *>(sh_scale);
        double acc[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) acc[t] = 0.0;
#pragma unroll 2
        for (int c = c0 + lane * 4; c < c1; c += 128) {
            float w[4], x[8][4];
            load4_plain<RT>(wrow, c, w);
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const int bt = min(b0 + t, B - 1);           // past the batch: the last token again (not stored)
                load4_plain<ACT>(reinterpret_cast<const uint8_t *>(hidden) + (size_t)bt * d * ab, c, x[t]);
            }
#pragma unroll
            for (int t = 0; t < 8; ++t)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[t] = fma((double)w[i], (double)x[t][i], acc[t]);
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            const double v = warp_sum(acc[t]);
            if (lane == t && b0 + t < B) lpart[((size_t)piece * B + b0 + t) * n_rows + row] = v;
        }
    }
}

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
// Dynamic shared memory: max(B * E + B, 16 * kRouteTok) doubles.
// JE: experts per lane in the gating (2, 4 or 8 for up to 64, 128, 256 experts): a kernel of its own
// for each, so that the gating code of a launch is one straight piece
// THREADS: kRouteThreads, or kRouteThreadsBig for the kernel of the larger batches (warp tasks only)
template <int ACT, int RT, int JE, int THREADS>
__device__ __forceinline__ void route_body(const Shape &sh, int B, const Workspace &ws, const void *__restrict__ hidden,
                                           const void *__restrict__ router, const void *__restrict__ sh_scale,
                                           const float *__restrict__ conf, int32_t *__restrict__ sel_idx,
                                           float *__restrict__ sel_w, int32_t *__restrict__ n_unique, const ZeroList &zl)
{
    extern __shared__ double s_dyn[];
    __shared__ int s_last;
    const int tid = threadIdx.x;
    // Programmatic dependent launch: everything this kernel writes is read by the previous
    // layer's kernels, so it waits for them first; the FFN kernel that follows may come up now
    // and do its own set-up (both instructions do nothing in a plain launch).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (zl.early && blockIdx.x == 0) {
        // the expert kernel of this layer polls these words from the moment it is scheduled, which is
        // after every block of this grid has passed the next instruction: they are cleared by then
        if (tid < 8) {
            asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(reinterpret_cast<unsigned long long *>(ws.early) + tid), "l"(0ull)
                         : "memory");
            __threadfence();
        }
        __syncthreads();
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // (block 0: where the arrival counter stood when the launch before had ended; see below)
    unsigned ticket_base = 0u;
    if (blockIdx.x == 0 && tid == 0)
        asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(ticket_base) : "l"(ws.ticket + 1) : "memory");
#pragma unroll
    for (int z = 0; z < 3; ++z) {
        uint4 *p = reinterpret_cast<uint4 *>(zl.ptr[z]);
        for (unsigned long long i = (unsigned long long)blockIdx.x * THREADS + tid; i < zl.n16[z];
             i += (unsigned long long)gridDim.x * THREADS)
            p[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    for (unsigned long long i = (unsigned long long)blockIdx.x * THREADS + tid; i < zl.perm_n16;
         i += (unsigned long long)gridDim.x * THREADS) {
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
    int n_arrive = 0;
    if (zl.ksplit > 0) {
        // larger batches: the logit pass as warp tasks over all blocks of the grid (a row block takes
        // 16 tokens per pass and its passes run one after the other: 22 us at 64 tokens)
        n_arrive = (int)gridDim.x;
        route_logit_tasks<ACT, RT>(sh, B, hidden, router, sh_scale, zl.lpart, zl.ksplit, (tid >> 5) * (int)gridDim.x + (int)blockIdx.x,
                                   (THREADS / 32) * (int)gridDim.x, tid & 31);
        __syncthreads();
    } else if constexpr (THREADS == kRouteThreads) {
    const int n_grp = zl.groups > 1 ? zl.groups : 1;
    n_arrive = n_rows * n_grp;
    // (early start of the expert kernel: it accumulates into what this grid clears as soon as the
    // list above is out, so the blocks that only clear arrive on the counter as well)
    if ((int)blockIdx.x >= n_arrive && !zl.early) return;
    if (zl.early) n_arrive = (int)gridDim.x;
    if ((int)blockIdx.x < n_rows * n_grp) {
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
    }
    }
    if (zl.early) __syncthreads();                        // all of this block's clearing, before its arrival
    // Block 0 runs the gating once every row has arrived (its SM tends to be the same from layer
    // to layer, so part of the gating code is still in its instruction cache: measured 0.6 % of
    // a layer against letting the last block to arrive do it).  Every block adds one arrival, with
    // release and acquire semantics by one thread, to a counter that is never reset; block 0
    // polls it, bounded, for the value it has when all blocks of THIS launch have arrived: the
    // value it will end on was left in the word behind the counter by the launch before (launches of
    // a context follow each other in stream order), and block 0 leaves the next one there, whether
    // its wait succeeded or not, since the late blocks still arrive.  So a wait that ran out poisons
    // nothing, and the waiting path is one atomic and one polled load, as short as it can be.  The
    // barriers on both sides extend the ordering to the block's other threads; the other blocks
    // wait for nothing.
    if (tid == 0) {
        unsigned target = 0u;
        if (blockIdx.x == 0) {
            target = ticket_base + (unsigned)n_arrive;
            asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(ws.ticket + 1), "r"(target) : "memory");
        }
        unsigned t;
        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(t) : "l"(ws.ticket) : "memory");
        int ok = 0;
        if (blockIdx.x == 0) {
            ok = (int)(t + 1u - target) >= 0 ? 1 : 0;
            for (unsigned i = 0; i < (1u << 22) && !ok; ++i) {
                unsigned v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ws.ticket) : "memory");
                if ((int)(v - target) >= 0) ok = 1;
                else __nanosleep(20);
            }
            if (!ok) atomicExch(ws.status, ST_TICKET_TIMEOUT);
        }
        s_last = ok;
    }
    __syncthreads();
    if (!s_last) return;
    gating_block<JE>(sh, B, ws, conf, sh_scale ? 1 : 0, sel_idx, sel_w, n_unique, s_dyn, zl.ksplit, zl.lpart, zl.early);
}

template <int ACT, int RT, int JE>
__global__ void __launch_bounds__(kRouteThreads)
route_kernel(Shape sh, int B, Workspace ws, const void *__restrict__ hidden, const void *__restrict__ router,
             const void *__restrict__ sh_scale, const float *__restrict__ conf, int32_t *__restrict__ sel_idx,
             float *__restrict__ sel_w, int32_t *__restrict__ n_unique, ZeroList zl)
{
    route_body<ACT, RT, JE, kRouteThreads>(sh, B, ws, hidden, router, sh_scale, conf, sel_idx, sel_w, n_unique, zl);
}

// The same with twice the warps, for the larger batches (logit pass by warp tasks only): the gating
// takes one warp per token, and at 64 tokens four passes of 16 warps were most of the kernel.
template <int ACT, int RT, int JE>
__global__ void __launch_bounds__(kRouteThreadsBig)
route_kernel_big(Shape sh, int B, Workspace ws, const void *__restrict__ hidden, const void *__restrict__ router,
                 const void *__restrict__ sh_scale, const float *__restrict__ conf, int32_t *__restrict__ sel_idx,
                 float *__restrict__ sel_w, int32_t *__restrict__ n_unique, ZeroList zl)
{
    route_body<ACT, RT, JE, kRouteThreadsBig>(sh, B, ws, hidden, router, sh_scale, conf, sel_idx, sel_w, n_unique, zl);
}

}  // namespace s2moe
