// The whole verification layer in ONE launch (kernel plan 4): the tcgen05 expert kernel of
// ffn_tc.cuh with a routing stage in front of its roles.
//
// Its CTAs first clear what the layer accumulates into and share the router's logit pass (a task
// is one router row x 8 tokens x one piece of the contraction, float64), meet once (a bounded
// grid-wide wait; one CTA per SM, all resident), and then eight warps of every CTA run the gating
// for themselves, all on the same numbers, while the producer and the MMA issuers already stream
// what needs no further routing decision, in two lots: first the shared experts and the expert of
// every token's largest logit (no bias of alpha <= 1 can push it out of that token's top-k), then,
// once E* and every token's first k experts by original logit are known, the experts of E* that
// are among some token's first k (at most their rank of others can pass them).  The unit tables
// therefore grow in three stages, and the accumulators of the early lots wait in tensor memory
// (up to eight buffers) until the gating has produced the token lists their epilogue needs.
// CTA 0 writes the layer's routing outputs.
//
// Measured on B200 against the two launches of plans 3 (routing kernel, then ffn_tc_kernel): slower
// on every workload here (OLMoE shape 56.7 against 49.8 us per layer, DeepSeek-V2-Lite shape 70.8
// against 63.4, Qwen1.5-MoE shape 64.2 against 57.6, Mixtral int4 167 against 140): inside the busy
// CTAs the gating takes two to three times as long as on a block of its own (its last table is
// ready 25 us after the kernel starts), and the epilogue warps that run it start draining the
// accumulators only then, which delays the first hand-over between the projections.  So the plan
// is offered on demand and the two-launch form stays the default.
//
// Everything that is the same in both kernels (PTX helpers, group table, tensor maps, the roles'
// inner loops) follows ffn_tc.cuh; the differences are the routing stage, the staged unit tables
// (more_units), the eight segments and the number of accumulator buffers.
#pragma once

#include "ffn_tc.cuh"
#include "gating.cuh"
#include "route.cuh"

namespace s2moe {
namespace fused {

struct TcPlan {
    int feasible;
    int n_cta;
    int stages;
    int stage_bytes;   // weight tile + token tiles, multiple of 1024
    int n1;            // tokens padded to 16 (phase-1 N)
    int tmem_cols;     // power of two >= 32
    int n_acc;         // accumulator buffers in tensor memory (runs the MMA issuers may be ahead of the epilogue)
    int n_iss;         // MMA issuer warps (2, or 4 on the int4 path when the accumulators fit)
    int tab_bytes;
    int x_bytes;       // > 0: the hidden states stay resident in shared memory (all k-tiles)
    int smem_bytes;
    int q4;            // block-int4 weights: packed tiles in the ring, dequantised into a second ring
    int a_stages;      // stages of that second ring
    int tok_off;       // offset of the token tiles inside a stage
    int kg;            // k-tiles per stage (1 for bf16 weights; 1, 2 or 4 for int4)
    int tokb;          // bytes of the token tiles of one k-tile
    int fused;         // the kernel also routes and gates (one launch per layer)
    int gate_bytes;    // fused: shared memory of the gating (staged logits and its tables)
    int ksplit;        // fused: pieces of the contraction a router row is cut into
};

// what the fused layer kernel needs for its routing stage (unused by the two-launch form)
struct TcRoute {
    const void *hidden, *router, *sh_scale;     // [B][d] bf16, [E][d] router dtype, [d] or NULL
    const float *conf;                          // [B] or NULL
    int32_t *sel_idx;                           // outputs of the layer call
    float *sel_w;
    int32_t *n_unique;
    double *lpart;                              // [ksplit][B][E (+1)] partial router logits
    unsigned long long *gbar;                   // arrivals of all launches so far (never reset)
    ZeroList zl;                                // what the kernel clears / copies before anything accumulates
    int early;                                  // the experts of the tokens' largest logits may start before the gating
};

struct TcArgs {
    Shape sh;
    Workspace ws;
    TcPlan plan;
    float *y;
    float *pre;                       // [gate|up][slot][f_g] fp32 pre-activations (zeroed by the routing stage)
    __nv_bfloat16 *act_hi, *act_lo;   // [slot][f_g]
    int B;
    TcRoute rt;
};

// warps of the fused kernel that run the gating while the layer starts: the four epilogue warps,
// the three converter warps and the watcher (they have nothing to do before the first accumulator
// is complete); their hardware barriers
constexpr int kTcGateWarps = 8, kTcGateBar = 2;

inline TcPlan tc_make_plan(const Shape &sh, int B, int n_sm, int n_slots)
{
    TcPlan p{};
    const int G = sh.E + sh.n_sh;
    p.n_cta = n_sm;
    p.n1 = (B + 15) & ~15;
    p.fused = 1;
    {
        p.gate_bytes = (int)((8 * ((size_t)B * sh.E + 2 * (size_t)B) + gate_mem_bytes(sh.E, B, sh.k) + 64 + 15) & ~(size_t)15);   // logits, confidences, gate logits, tables
        // a router row is cut into pieces so that the warps of all CTAs share the logit pass
        const int rows = sh.E + 1, tgs = (B + 7) / 8, warps = n_sm * 11;
        int ks = warps / (rows * tgs);
        if (ks > 8) ks = 8;
        if (ks > sh.d / 128) ks = sh.d / 128;
        p.ksplit = ks < 1 ? 1 : ks;
    }
    // token area of a stage: phase 1 = n1 rows of 128 bytes; phase 2 = per 8 slots their hi rows
    // (1 KiB) and right behind them their lo rows (a group never has more tokens than B)
    p.stage_bytes = kTcWTile + 2048 * ((B + 7) / 8);
    p.stage_bytes = (p.stage_bytes + 1023) & ~1023;
    p.tab_bytes = ((int)sizeof(TcGroup) * (G + 1) + 8 * n_slots + 4 * (G + 2) + p.gate_bytes + 1023) & ~1023;
    // The ring is what keeps HBM busy (bytes in flight = stages x 16 KiB per SM, against a loaded
    // latency of 2-3 us), so shared memory goes to stages first: the hidden-state tiles stay
    // resident only if the ring reaches its maximum depth anyway, otherwise every stage fetches
    // its token k-tile (2 KiB per 16 tokens, an L2 hit) next to the weight k-tile.
    p.x_bytes = ((sh.d + 63) / 64) * p.n1 * 128;
    if ((kTcMaxSmem - p.tab_bytes - 1024 - p.x_bytes) / p.stage_bytes < kTcMaxStages) p.x_bytes = 0;
    p.stages = (kTcMaxSmem - p.tab_bytes - 1024 - p.x_bytes) / p.stage_bytes;
    if (p.stages > kTcMaxStages) p.stages = kTcMaxStages;
    p.n_iss = 2;
    // accumulators: buffers x 2 issuers x up to 2 * n1 columns.  Two buffers keep the issuers busy while
    // the epilogue drains; the fused kernel takes as many as tensor memory holds (up to 8), because
    // there the accumulators of the early groups cannot be drained before the gating has finished
    p.n_acc = 2;
    {
        p.n_acc = 512 / (4 * p.n1);
        if (p.n_acc > 8) p.n_acc = 8;
        if (p.n_acc < 2) p.n_acc = 2;
    }
    p.tmem_cols = 32;
    while (p.tmem_cols < p.n_acc * 4 * p.n1) p.tmem_cols <<= 1;
    p.smem_bytes = p.tab_bytes + p.x_bytes + p.stages * p.stage_bytes + 1024;   // + slack to align to 1024
    p.tok_off = kTcWTile;
    p.kg = 1;
    p.tokb = 2048 * ((B + 7) / 8);
    p.feasible = p.stages >= 4 && B <= kMaxTokens && sh.weight_dtype == DT_BF16 && sh.act_dtype == DT_BF16 &&
                 sh.d % 64 == 0;
    if (sh.weight_dtype == DT_Q4B32) {
        // a stage holds the packed k-tiles and their unit's scales; the TMA copy of the scales
        // wants rows of a multiple of 16 bytes, i.e. contraction lengths of 256.
        // A packed k-tile is only 4 KiB, so a stage carries four of them (a whole unit): one
        // TMA copy, one hand-over to the tensor core and one release per stage instead of four.
        p.q4 = 1;
        p.x_bytes = 0;
        const int budget = kTcMaxSmem - p.tab_bytes - 1024;
        // The dequantised tiles live in tensor memory (A operand of the MMAs): columns 256..511 hold
        // two slots of a whole unit (4 k-tiles x 32 columns of bf16 pairs), columns 0..255 the
        // accumulators: 2 buffers x issuers x 2 * n1 columns.  Issuing is what has to keep up with
        // a stage that is cheap to fetch, so as many issuers as the accumulators leave room for.
        p.n_iss = 16 * p.n1 <= kTcQ4ACol ? 4 : (8 * p.n1 <= kTcQ4ACol ? 2 : 1);
        p.tmem_cols = 512;
        p.n_acc = 2;
        // The token tiles of a stage do not travel with its packed tiles: they are fetched into a
        // slot that belongs to the ring of dequantised tiles, just before they are used, so that a
        // stage is free again as soon as the dequantising warps have read it (its life decides
        // how many bytes are in flight) and not only when the MMAs have completed.
        p.kg = kTcQ4KG;
        p.tok_off = p.kg * kTcQ4Packed + kTcQ4Scales;
        p.stage_bytes = (p.tok_off + 1023) & ~1023;
        p.a_stages = 2;
        p.stages = (budget - p.a_stages * p.kg * p.tokb) / p.stage_bytes;
        if (p.stages > kTcMaxStages) p.stages = kTcMaxStages;
        p.smem_bytes = p.tab_bytes + p.stages * p.stage_bytes + p.a_stages * p.kg * p.tokb + 1024;
        p.feasible = p.stages >= 3 && B <= kMaxTokens && sh.act_dtype == DT_BF16 && sh.d % 256 == 0 &&
                     sh.f % 256 == 0 && (sh.n_sh == 0 || sh.f_sh % 256 == 0);
    }
    return p;
}

// units of a group: phase 1 = 2 matrices x row blocks x k-pieces, phase 2 = row blocks x k-pieces

// ---- routing stage of the fused kernel ------------------------------------------------------

struct TcUnit {                        // plain ints: the single-thread roles read these on their critical path
    int phase, a, mat, rb, kt0, kt1;   // group slot, matrix (0 gate, 1 up, 2 down), row block, k-tile range
    int n;                             // MMA N: phase 1 tokens padded to 16; phase 2 16 per 8 slots (hi | lo)
    int first, last;                   // first / last unit of an accumulation run (see the kernel)
    int wave;                          // 0 / 1: the group belongs to the first / second wave
};
static_assert(sizeof(TcUnit) == 40, "layout");

__device__ __forceinline__ TcUnit lt_decode(const TcGroup *groups, int n_active, int total1, int u, int d, int n1)
{
    TcUnit t;
    if (u < total1) {
        t.phase = 1;
        t.a = upper_group1(groups, n_active, u);
        const TcGroup &g = groups[t.a];
        const int local = u - g.p1, kp = tc_kpieces(d), rbs = (g.f + 127) / 128;
        const int piece = local % kp, rest = local / kp;
        t.rb = rest % rbs;
        t.mat = rest / rbs;
        t.kt0 = piece * kTcKT;
        t.kt1 = min((d + 63) / 64, t.kt0 + kTcKT);
        t.n = n1;
    } else {
        t.phase = 2;
        const int v = u - total1;
        t.a = upper_group2(groups, n_active, v);
        const TcGroup &g = groups[t.a];
        const int local = v - g.p2, kp = tc_kpieces(g.f);
        const int piece = local % kp;
        t.rb = local / kp;
        t.mat = 2;
        t.kt0 = piece * kTcKT;
        t.kt1 = min((g.f + 63) / 64, t.kt0 + kTcKT);
        t.n = 16 * ((g.T + 7) / 8);
    }
    return t;
}

// first | last << 1 | (phase == 2) << 2 | n << 8: the single-thread roles share their schedulers with
// busy warps, so every instruction they do not need per unit counts
__device__ __forceinline__ uint32_t lt_unit_meta(const TcUnit &t)
{
    return (uint32_t)t.first | ((uint32_t)t.last << 1) | ((t.phase == 2 ? 1u : 0u) << 2) | ((uint32_t)t.n << 8);
}

// The share of one CTA in the eight segments of a layer (see the kernel): per segment the first
// unit, the number of units and the half-unit trim bits.
constexpr int kTcSegs = 8;
struct TcShare {
    int start[kTcSegs], cnt[kTcSegs], trim[kTcSegs];
};

// Every CTA takes one contiguous run of units of each segment (sizes differ by at most one; the
// CTAs that get the extra unit rotate from segment to segment, so the totals differ by at most
// one as well).  Where every unit of a projection has all its four k-tiles (contraction length a
// multiple of 256) the segments are dealt in half units, so that the CTAs of a segment differ by
// two k-tiles (0.75 us) instead of four: a share may then begin with the second half of a unit and
// end with the first half of one (trim bits 1 and 2).  Measured at the OLMoE shape: 0.7 % of a
// layer; dealing single k-tiles cuts more accumulation runs in two and gives it back.
// bound[0..6]: the segments' boundaries in the numbering of lt_decode.
__device__ __forceinline__ void lt_shares(const int (&bound)[kTcSegs + 1], bool halves1, bool halves2, int P, int cta, TcShare &out)
{
    int rot = 0;
#pragma unroll
    for (int sg = 0; sg < kTcSegs; ++sg) {
        const bool halves = sg < 6 ? halves1 : halves2;
        const int begin = bound[sg], n = bound[sg + 1] - bound[sg];
        if (n <= 0) { out.cnt[sg] = 0; out.start[sg] = begin; out.trim[sg] = 0; continue; }
        const int m = halves ? 2 : 1, n2 = n * m;
        const int q = n2 / P, r = n2 - q * P;
        int c = cta - rot;                             // (cta - rot) mod P without a division
        if (c < 0) c += P;
        const int cnt2 = q + (c < r ? 1 : 0), start2 = c * q + min(c, r);
        const int u0 = halves ? start2 >> 1 : start2, u1 = halves ? (start2 + cnt2 - 1) >> 1 : start2 + cnt2 - 1;
        out.cnt[sg] = cnt2 > 0 ? u1 - u0 + 1 : 0;
        out.start[sg] = begin + u0;
        out.trim[sg] = (halves && cnt2 > 0) ? ((start2 & 1) | (((start2 + cnt2) & 1) << 1)) : 0;
        rot += r;
        if (rot >= P) rot -= P;
    }
}

// unit i of a CTA's sequence (segments in order)
__device__ __forceinline__ TcUnit lt_unit_make(const TcShare &shr, const TcGroup *groups, int n_groups, int total1, int a_split,
                                               int i, int d, int n1)
{
    // (static indices only: the shares stay in registers)
    int seg = 0, j = i, start = shr.start[0], cnt = shr.cnt[0], trim = shr.trim[0];
#pragma unroll
    for (int sg = 1; sg < kTcSegs; ++sg)
        if (seg == sg - 1 && j >= cnt) { j -= cnt; seg = sg; start = shr.start[sg]; cnt = shr.cnt[sg]; trim = shr.trim[sg]; }
    TcUnit t = lt_decode(groups, n_groups, total1, start + j, d, n1);
    const int K = t.phase == 1 ? d : groups[t.a].f;
    if (j == 0 && (trim & 1)) t.kt0 += kTcKT / 2;            // the CTA before this one has the first half
    if (j == cnt - 1 && (trim & 2)) t.kt1 -= kTcKT / 2;      // the next CTA has the second half
    t.wave = t.a >= a_split ? 1 : 0;
    t.first = (j == 0 || t.kt0 == 0) ? 1 : 0;
    t.last = (j == cnt - 1 || t.kt1 == (K + 63) / 64) ? 1 : 0;
    return t;
}

// The layer kernel (see the head of this file).
template <bool Q4>
__global__ void __launch_bounds__(Q4 ? kTcQ4Threads : kTcThreads, 1)
layer_tc_kernel(const __grid_constant__ TcMaps maps, TcArgs p)
{
    extern __shared__ __align__(1024) uint8_t tc_smem[];
    __shared__ __align__(8) uint64_t full_bar[kTcMaxStages], empty_bar[kTcMaxStages];
    __shared__ __align__(8) uint64_t acc_full[8], acc_empty[8], ep_bar, x_bar, cv_bar, conv_go[2];
    __shared__ __align__(8) uint64_t a_full[kTcMaxAStages], a_empty[kTcMaxAStages];   // int4: dequantised tiles
    __shared__ uint32_t s_tmem;
    __shared__ int s_flag, s_go;
    __shared__ TcUnit s_units[kTcMaxUnits];
    __shared__ uint32_t s_umeta[kTcMaxUnits];      // what an MMA issuer needs of a unit, in one word (lt_unit_meta)
    __shared__ volatile int s_ready[2];            // wave w's activations are written (set by the watcher warp)
    // the unit tables come in three stages in the fused kernel: s_tab = 1 when this CTA's units of the
    // first lot of early groups are decoded (s_nunits[0] units), 2 with the second lot (s_nunits[1]),
    // 3 when everything is (s_nunits[2]); the two-launch form starts at 3
    __shared__ volatile int s_tab;
    __shared__ int s_nunits[3];
    __shared__ TcShare s_share;
    __shared__ int s_nact, s_split, s_total1;      // active groups, first group of wave 1 (s_nact: one wave), phase-1 units
    __shared__ unsigned s_lot[3][8];               // fused: experts of the first and second early lot, all selected experts (bit words)

    const Shape &sh = p.sh;
    const Workspace &ws = p.ws;
    const TcPlan &pl = p.plan;
    const int NI = Q4 ? p.plan.n_iss : 2;          // MMA issuers: a compile-time 2 on the bf16 path
    const int NACC = p.plan.n_acc;                 // accumulator buffers
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // programmatic dependent launch: whatever is in front of this grid in the stream (the previous
    // layer) must have finished before this layer's buffers are cleared
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int n_slots = p.B * sh.k + sh.n_sh * p.B;          // every token fills k routed slots
    const int G = sh.E + sh.n_sh;
    const int S = pl.stages;
    const int P = gridDim.x;

    TcGroup *groups = reinterpret_cast<TcGroup *>(tc_smem);
    int *s_epfx = reinterpret_cast<int *>(tc_smem + sizeof(TcGroup) * (G + 1));     // [n_active + 1] activation elements in front of a group, in group order
    int *s_slot_token = s_epfx + (G + 2);
    float *s_slot_w = reinterpret_cast<float *>(s_slot_token + n_slots);
    uint8_t *gate_area = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(s_slot_w + n_slots) + 15) & ~(uintptr_t)15);
    uint8_t *xres = tc_smem + pl.tab_bytes;
    xres = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(xres) + 1023) & ~(uintptr_t)1023);
    uint8_t *ring = xres + pl.x_bytes;
    uint8_t *tokring = ring + (size_t)pl.stages * pl.stage_bytes;    // int4 only: token tiles, one slot per slot of dequantised tiles

    const int u1r = tc_units1(sh.f, sh.d), u2r = tc_units2(sh.f, sh.d);
    const int u1s = sh.n_sh ? tc_units1(sh.f_sh, sh.d) : 0, u2s = sh.n_sh ? tc_units2(sh.f_sh, sh.d) : 0;
    // segments are dealt in half units where every unit has all its k-tiles; the int4 path needs whole units
    const bool halves1 = !Q4 && sh.d % 256 == 0;
    const bool halves2 = !Q4 && sh.f % 256 == 0 && (sh.n_sh == 0 || sh.f_sh % 256 == 0);

    if (tid == 0) {
        s_ready[0] = 0;
        s_ready[1] = 0;
        s_tab = 0;
        s_go = 1;
    }
    if (warp == 2) {
        // barrier set-up, spread over a warp so that it runs beside the work of the others
        if (lane < pl.stages) {
            mbar_init(&full_bar[lane], 1);
            mbar_init(&empty_bar[lane], Q4 ? kTcQ4DeqWarps : NI);   // one commit from each MMA issuer; int4: the dequantising warps
        }
        if (lane < pl.n_acc) {
            mbar_init(&acc_full[lane], NI);
            mbar_init(&acc_empty[lane], 4);
        }
        if (lane < 2) mbar_init(&conv_go[lane], 4);
        if (Q4 && lane < pl.a_stages) {
            mbar_init(&a_full[lane], kTcQ4DeqWarps + 1);   // the dequantising warps and the producer's arrival with the token bytes
            mbar_init(&a_empty[lane], NI);
        }
        if (lane == 0) {
            mbar_init(&ep_bar, 4);
            mbar_init(&x_bar, 1);
            mbar_init(&cv_bar, 3);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // TMEM: accumulators of two runs for each of the two issuers
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                     "r"((uint32_t)pl.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    {
        const TcRoute &rt = p.rt;
        // ---- clear what the layer accumulates into (and, int4, leave the binary16 column-permuted
        // copy of the hidden states): every CTA its share, all of it before the grid-wide meeting
        {
            const unsigned long long gt = (unsigned long long)blockIdx.x * blockDim.x + tid, gn = (unsigned long long)P * blockDim.x;
#pragma unroll
            for (int z = 0; z < 3; ++z) {
                uint4 *q = reinterpret_cast<uint4 *>(rt.zl.ptr[z]);
                for (unsigned long long i = gt; i < rt.zl.n16[z]; i += gn) q[i] = make_uint4(0u, 0u, 0u, 0u);
            }
            for (unsigned long long i = gt; i < rt.zl.perm_n16; i += gn) {
                const uint4 v = rt.zl.perm_src[i];             // halves h0..h7 (bf16)
                rt.zl.perm_dst[i] = make_uint4(bf16x2_to_f16x2(__byte_perm(v.x, v.z, 0x5410)), bf16x2_to_f16x2(__byte_perm(v.x, v.z, 0x7632)),
                                               bf16x2_to_f16x2(__byte_perm(v.y, v.w, 0x5410)), bf16x2_to_f16x2(__byte_perm(v.y, v.w, 0x7632)));
            }
            if (Q4) asm volatile("fence.proxy.async.global;" ::: "memory");   // the copy is read by TMA copies of all CTAs
        }
        // ---- the logit pass, shared by the warps of all CTAs
        {
            const int nwarps = (int)blockDim.x >> 5;
            if (sh.router_dtype == DT_F32)
                route_logit_tasks<DT_BF16, DT_F32>(sh, p.B, rt.hidden, rt.router, rt.sh_scale, rt.lpart, pl.ksplit, warp * P + (int)blockIdx.x, nwarps * P, lane);
            else
                route_logit_tasks<DT_BF16, DT_BF16>(sh, p.B, rt.hidden, rt.router, rt.sh_scale, rt.lpart, pl.ksplit, warp * P + (int)blockIdx.x, nwarps * P, lane);
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        // ---- the meeting: every CTA adds one arrival to a counter that is never reset (all launches
        // of a context have the same grid, so a launch ends on a multiple of the grid size) and
        // waits, bounded, for that multiple.  A wait that gave up leaves nothing behind: the others
        // still arrive.  The barriers on both sides extend the ordering to the block's threads.
        if (tid == 0) {
            unsigned long long t;
            asm volatile("atom.add.acq_rel.gpu.global.u64 %0, [%1], 1;" : "=l"(t) : "l"(rt.gbar) : "memory");
            const unsigned long long target = (t / (unsigned long long)P + 1ull) * (unsigned long long)P;
            int ok = t + 1ull == target ? 1 : 0;
            for (unsigned i = 0; i < kTcSpinLimit && !ok; ++i) {
                unsigned long long v;
                asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(rt.gbar) : "memory");
                if (v >= target) ok = 1;
                else __nanosleep(32);
            }
            if (!ok) atomicExch(ws.status, ST_TICKET_TIMEOUT);
            s_go = ok;
        }
        __syncthreads();
    }
    const uint32_t tmem_base = s_tmem;
    const bool go = s_go != 0;

    // Eight segments in time order.  Phase 1 comes in up to three lots as the routing becomes known
    // (fused kernel only: first the shared experts and the expert of every token's largest logit,
    // then the experts that are in E* and among some token's first k, then the rest; the two-launch
    // form has the last lot only), and every lot is cut in two at the group that brings it to the
    // wave share, so that wherever the boundary between wave 0 and wave 1 finally falls it is a
    // boundary between segments; then phase 2 of wave 0 and of wave 1.  Every segment is dealt over
    // all CTAs.  Contiguous units are consecutive k-pieces of one 128-row block, so a CTA
    // accumulates them in one TMEM accumulator and the epilogue runs once per run of k-pieces
    // instead of once per unit; only row blocks cut by a CTA boundary are reduced from two CTAs.
    const bool gate_warp = (warp >= 2 && warp <= 5) || (warp >= 7 && warp <= 10);
    // first phase-1 / phase-2 unit of the group at position a of the fused kernel's group order
    // (the shared experts first, then routed experts)
    auto p1_of = [&](int a) -> int { return a < sh.n_sh ? a * u1s : sh.n_sh * u1s + (a - sh.n_sh) * u1r; };
    auto p2_of = [&](int a) -> int { return a < sh.n_sh ? a * u2s : sh.n_sh * u2s + (a - sh.n_sh) * u2r; };
    // the group in [max(lo, 1), hi] whose first unit comes closest to the wave share of `total` (hi when
    // the range is empty): where a lot of groups is cut in two
    auto cut_at = [&](int lo, int hi, int total) -> int {
        int best_a = hi;
        long long best = -1;
        for (int a = lo < 1 ? 1 : lo; a <= hi; ++a) {
            long long dist = (long long)p1_of(a) * kTcSplitDen - (long long)total * kTcSplitNum;
            if (dist < 0) dist = -dist;
            if (best < 0 || dist < best) { best = dist; best_a = a; }
        }
        return best_a;
    };
    if (go && gate_warp) {
        const TcRoute &rt = p.rt;
        const int gw = warp <= 5 ? warp - 2 : warp - 3;            // 0..7 inside the gating group
        const GateGroup gg{gw * 32 + lane, kTcGateWarps * 32, kTcGateBar};
        const int E = sh.E, B = p.B, k = sh.k, n_rows = E + (rt.sh_scale ? 1 : 0), n_routed = B * k;
        const int EW = (E + 31) >> 5;                              // bit words of an expert set
        double *s_l = reinterpret_cast<double *>(gate_area), *s_w = s_l + B * E, *s_gl = s_w + B;   // logits, confidences, gate logits
        const GateMem gm = gate_mem_carve(s_gl + B, E, B, k);
        const bool bias_on = sh.alpha > 0.0 && sh.cap < E && k < E;
        // ---- stage the logits: the pieces of a row added in ascending order (all loads first)
#pragma unroll 1
        for (int i = gg.t; i < B * n_rows; i += gg.n) {
            const int b = i / n_rows, r = i - b * n_rows;
            double v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = q < pl.ksplit ? __ldcg(&rt.lpart[((size_t)q * B + b) * n_rows + r]) : 0.0;
            double acc = v[0];
#pragma unroll
            for (int q = 1; q < 8; ++q) acc += v[q];
            if (r < E) s_l[b * E + r] = acc;
            else s_gl[b] = acc;
        }
#pragma unroll 1
        for (int b = gg.t; b < B; b += gg.n) s_w[b] = rt.conf ? (double)rt.conf[b] : 1.0;
        if (gg.t < 24) s_lot[gg.t >> 3][gg.t & 7] = 0u;
        for (int e = gg.t; e < E; e += gg.n) gm.star[e] = 0;
        if (gg.t < 8) gm.star32[gg.t] = 0u;
        gate_sync(gg);
        // ---- first lot of early groups: the shared experts, and (alpha <= 1) every token's first
        // expert in the order (logit descending, id ascending), which no bias can push out of its
        // top-k: six warps; the other two find E* meanwhile
        if (gw < 2) {
            if (bias_on) gating_estar(sh, B, s_l, s_w, gm, gg.t, 64, kTcGateBar + 1);
        } else if (rt.early) {
#pragma unroll 1
            for (int b = gw - 2; b < B; b += kTcGateWarps - 2) {
                unsigned long long best = 0ull;
                int be = 0;
                for (int e = lane; e < E; e += 32) {
                    const unsigned long long ke = dkey(s_l[b * E + e]);
                    if (ke > best) { best = ke; be = e; }
                }
                const unsigned hb = warp_max_holders(best, best != 0ull);
                const unsigned me = __reduce_min_sync(0xffffffffu, ((hb >> lane) & 1u) ? (unsigned)be : 0xffffffffu);
                if (lane == 0) atomicOr(&s_lot[0][me >> 5], 1u << (me & 31));
            }
        }
        gate_sync(gg);
        // position of expert e among the members of a bit set
        auto set_rank = [&](const unsigned *set, int e) -> int {
            int r = __popc(set[e >> 5] & ((1u << (e & 31)) - 1u));
            for (int w = 0; w < (e >> 5); ++w) r += __popc(set[w]);
            return r;
        };
        auto set_size = [&](const unsigned *set) -> int {
            int n = 0;
            for (int w = 0; w < EW; ++w) n += __popc(set[w]);
            return n;
        };
        const int n_a = set_size(s_lot[0]);                        // experts of the first lot
        {
            // group entries of the first lot: the shared experts, then its experts in ascending order
            for (int a = gg.t; a < sh.n_sh; a += gg.n) {
                TcGroup gr{};
                gr.group = E + a; gr.f = sh.f_sh; gr.p1 = a * u1s; gr.p2 = a * u2s;
                groups[a] = gr;
            }
            for (int e = gg.t; e < E; e += gg.n) {
                if ((s_lot[0][e >> 5] >> (e & 31)) & 1u) {
                    const int r = set_rank(s_lot[0], e);
                    TcGroup gr{};
                    gr.group = e; gr.f = sh.f; gr.p1 = sh.n_sh * u1s + r * u1r; gr.p2 = sh.n_sh * u2s + r * u2r;
                    groups[sh.n_sh + r] = gr;
                }
            }
            if (gg.t == 0) {
                const int e1 = p1_of(sh.n_sh + n_a), b1 = p1_of(cut_at(0, sh.n_sh + n_a, e1));
                const int bound[kTcSegs + 1] = {0, b1, e1, e1, e1, e1, e1, e1, e1};
                TcShare shr;
                lt_shares(bound, halves1, halves2, P, (int)blockIdx.x, shr);
                s_share = shr;
                s_nunits[0] = shr.cnt[0] + shr.cnt[1];
                // what a unit beyond the decoded table is made from (see unit_at): for now the early
                // groups alone; the final values replace these once the groups are complete, and an
                // early unit decodes the same from either
                s_nact = sh.n_sh + n_a;
                s_total1 = 0x7fffffff;
                s_split = 0x7fffffff;
            }
        }
        gate_sync(gg);
        for (int i = gg.t; i < s_nunits[0] && i < kTcMaxUnits; i += gg.n) {
            const TcUnit t = lt_unit_make(s_share, groups, sh.n_sh + n_a, 0x7fffffff, 0x7fffffff, i, sh.d, pl.n1);
            s_units[i] = t;
            s_umeta[i] = lt_unit_meta(t);
        }
        __threadfence_block();
        gate_sync(gg);
        if (gg.t == 0) s_tab = 1;
        // ---- the gating, first part: E*, lambda_b, every token's first k experts by original logit
        if (E <= 64) gating_part1<2>(sh, B, s_l, s_w, gg, gm, false, true, true);
        else if (E <= 128) gating_part1<4>(sh, B, s_l, s_w, gg, gm, false, true, true);
        else gating_part1<8>(sh, B, s_l, s_w, gg, gm, false, true, true);
        // ---- second lot of early groups: an expert of E* that is among a token's first k stays in that
        // token's top-k whatever the bias does to the others (at most its rank of them pass it), so
        // E* intersected with the union of the tokens' first k can start now
        if (bias_on && rt.early) {
            const int J = E <= 64 ? 2 : (E <= 128 ? 4 : 8);
            for (int i = gg.t; i < B * J; i += gg.n) {
                const int j = i % J;
                const unsigned wd = gm.topk[i] & gm.star32[j] & ~s_lot[0][j];
                if (wd) atomicOr(&s_lot[1][j], wd);
            }
        }
        gate_sync(gg);
        const int n_b = set_size(s_lot[1]), n_early = sh.n_sh + n_a + n_b;
        {
            for (int e = gg.t; e < E; e += gg.n) {
                if ((s_lot[1][e >> 5] >> (e & 31)) & 1u) {
                    const int a = sh.n_sh + n_a + set_rank(s_lot[1], e);
                    TcGroup gr{};
                    gr.group = e; gr.f = sh.f; gr.p1 = sh.n_sh * u1s + (a - sh.n_sh) * u1r; gr.p2 = sh.n_sh * u2s + (a - sh.n_sh) * u2r;
                    groups[a] = gr;
                }
            }
            if (gg.t == 0) {
                const int m1 = sh.n_sh + n_a, e1 = p1_of(m1), b1 = p1_of(cut_at(0, m1, e1));
                const int e2 = p1_of(n_early), b3 = p1_of(cut_at(m1, n_early, e2));
                const int bound[kTcSegs + 1] = {0, b1, e1, b3, e2, e2, e2, e2, e2};
                TcShare shr;
                lt_shares(bound, halves1, halves2, P, (int)blockIdx.x, shr);
                s_share = shr;                         // (the first two segments come out as before)
                s_nunits[1] = shr.cnt[0] + shr.cnt[1] + shr.cnt[2] + shr.cnt[3];
            }
        }
        __threadfence_block();
        gate_sync(gg);
        if (gg.t == 0) s_nact = n_early;               // the second lot's groups are complete
        for (int i = s_nunits[0] + gg.t; i < s_nunits[1] && i < kTcMaxUnits; i += gg.n) {
            const TcUnit t = lt_unit_make(s_share, groups, n_early, 0x7fffffff, 0x7fffffff, i, sh.d, pl.n1);
            s_units[i] = t;
            s_umeta[i] = lt_unit_meta(t);
        }
        __threadfence_block();
        gate_sync(gg);
        if (gg.t == 0) s_tab = 2;
        // ---- the gating, second part; CTA 0 also writes the call's outputs
        const bool writer = blockIdx.x == 0;
        if (E <= 64) gating_part2<2>(sh, B, s_l, gg, gm, writer ? rt.sel_idx : nullptr, writer ? rt.sel_w : nullptr, false);
        else if (E <= 128) gating_part2<4>(sh, B, s_l, gg, gm, writer ? rt.sel_idx : nullptr, writer ? rt.sel_w : nullptr, false);
        else gating_part2<8>(sh, B, s_l, gg, gm, writer ? rt.sel_idx : nullptr, writer ? rt.sel_w : nullptr, false);
        // ---- the tables in their final form.  Group order: the early groups, then the other selected
        // experts in ascending order; slots stay in expert order (routed first, then shared).
        const int U = *gm.U, n_active = U + sh.n_sh;
        {
            // all selected experts as a bit set, one ballot per 32 experts
            for (int e0 = gw * 32; e0 < E; e0 += kTcGateWarps * 32) {
                const unsigned wd = __ballot_sync(0xffffffffu, e0 + lane < E && gm.cnt[e0 + lane] > 0);
                if (lane == 0) s_lot[2][e0 >> 5] = wd;
            }
        }
        gate_sync(gg);
        const unsigned long long all = B >= 64 ? ~0ull : ((1ull << B) - 1ull);
        for (int e = gg.t; e < E; e += gg.n) {
            if (gm.cnt[e] == 0) continue;
            const bool in_a = (s_lot[0][e >> 5] >> (e & 31)) & 1u, in_b = (s_lot[1][e >> 5] >> (e & 31)) & 1u;
            int a;
            if (in_a) a = sh.n_sh + set_rank(s_lot[0], e);
            else if (in_b) a = sh.n_sh + n_a + set_rank(s_lot[1], e);
            else {
                // position among the selected experts outside both lots
                int r = __popc(s_lot[2][e >> 5] & ~s_lot[0][e >> 5] & ~s_lot[1][e >> 5] & ((1u << (e & 31)) - 1u));
                for (int w = 0; w < (e >> 5); ++w) r += __popc(s_lot[2][w] & ~s_lot[0][w] & ~s_lot[1][w]);
                a = n_early + r;
            }
            TcGroup gr;
            gr.group = e; gr.T = gm.cnt[e]; gr.off = gm.off[e]; gr.f = sh.f; gr.mask = gm.mask[e];
            gr.p1 = sh.n_sh * u1s + (a - sh.n_sh) * u1r;
            gr.p2 = sh.n_sh * u2s + (a - sh.n_sh) * u2r;
            groups[a] = gr;
        }
        for (int a = gg.t; a < sh.n_sh; a += gg.n) {
            TcGroup gr;
            gr.group = E + a; gr.T = B; gr.off = n_routed + a * B; gr.f = sh.f_sh; gr.mask = all;
            gr.p1 = a * u1s; gr.p2 = a * u2s;
            groups[a] = gr;
        }
        const int total1 = sh.n_sh * u1s + U * u1r, total2 = sh.n_sh * u2s + U * u2r;
        // The boundary between the waves: of the segment boundaries inside phase 1 (the cut and the end
        // of either early lot, the cut of the rest) the one that comes closest to the wave share.
        const int m1 = sh.n_sh + n_a, e1 = p1_of(m1), x_a = cut_at(0, m1, e1);
        const int e2 = p1_of(n_early), x_b = cut_at(m1, n_early, e2);
        const int x_r = cut_at(n_early, n_active, total1);
        int sp = n_active;
        {
            const int cand[5] = {x_a, m1, x_b, n_early, x_r};
            long long best = -1;
#pragma unroll
            for (int c = 0; c < 5; ++c) {
                const int a = cand[c];
                if (a < 1 || a > n_active - 1) continue;           // both waves keep at least one group
                long long dist = (long long)p1_of(a) * kTcSplitDen - (long long)total1 * kTcSplitNum;
                if (dist < 0) dist = -dist;
                if (best < 0 || dist < best) { best = dist; sp = a; }
            }
        }
        if (gg.t == 0) {
            const int b5 = p1_of(x_r);
            const int split2 = sp < n_active ? p2_of(sp) : total2;
            const int bound[kTcSegs + 1] = {0, p1_of(x_a), e1, p1_of(x_b), e2, b5, total1, total1 + split2, total1 + total2};
            TcShare shr;
            lt_shares(bound, halves1, halves2, P, (int)blockIdx.x, shr);
            s_share = shr;
            int n = 0;
            for (int sg = 0; sg < kTcSegs; ++sg) n += shr.cnt[sg];
            s_nunits[2] = n;
        }
        __threadfence_block();
        gate_sync(gg);
        if (gg.t == 0) {                               // the groups are complete before their number grows
            s_split = sp;
            s_total1 = total1;
            s_nact = n_active;
        }
        for (int i = s_nunits[1] + gg.t; i < s_nunits[2] && i < kTcMaxUnits; i += gg.n) {
            const TcUnit t = lt_unit_make(s_share, groups, n_active, total1, sp, i, sh.d, pl.n1);
            s_units[i] = t;
            s_umeta[i] = lt_unit_meta(t);
        }
        __threadfence_block();
        gate_sync(gg);
        if (gg.t == 0) s_tab = 3;
        // ---- what only these warps' later roles need: slots (tokens ascending inside an expert, the
        // shared experts' slots behind the routed ones) and the groups' element ranges
        for (int i = gg.t; i < n_routed; i += gg.n) {
            const int b = i / k, e = gm.sel[i];
            const int pos = gm.off[e] + __popcll(gm.mask[e] & ((1ull << b) - 1ull));
            s_slot_token[pos] = b;
            s_slot_w[pos] = gm.pw[i];
        }
        for (int i = gg.t; i < sh.n_sh * B; i += gg.n) {
            const int b = i % B;
            s_slot_token[n_routed + i] = b;
            s_slot_w[n_routed + i] = rt.sh_scale ? (float)(1.0 / (1.0 + exp_once(-s_gl[b]))) : 1.0f;
        }
        if (gg.t == 0) {
            int acc = 0;
            for (int a = 0; a < n_active; ++a) { s_epfx[a] = acc; acc += groups[a].T * groups[a].f; }
            s_epfx[n_active] = acc;
        }
        if (writer) {
            // the layer's routing outputs and the bucketing arrays in the workspace (debug reads)
            Workspace wsw = ws;
            wsw.gtab = nullptr;
            for (int b = gg.t; b < B; b += gg.n) ws.gate_logit[b] = s_gl[b];
            for (int i = gg.t; i < B * E; i += gg.n) ws.logits[i] = s_l[i];
            gate_sync(gg);
            Shape shw = sh;
            shw.plan = 3;
            gating_writeout(shw, B, wsw, gm, rt.sh_scale ? 1 : 0, rt.n_unique, gg);
        }
        gate_sync(gg);
    }

    // the unit table as far as it is known to this thread, and a wait for more of it
    int tab_seen = 0, n_known = 0;
    // 1: unit i exists, 0: the sequence has ended, -1: the wait for the tables gave up
    auto more_units = [&](int i) -> int {
        while (i >= n_known) {
            if (tab_seen == 3) return 0;
            bool ok = false;
            for (unsigned spin = 0; spin < kTcSpinLimit; ++spin) {
                if (s_tab > tab_seen) { ok = true; break; }
                __nanosleep(40);
            }
            if (!ok) return -1;
            tab_seen = s_tab;
            __threadfence_block();
            n_known = s_nunits[tab_seen - 1];
        }
        return 1;
    };
    auto unit_at = [&](int i) -> TcUnit {
        return i < kTcMaxUnits ? s_units[i] : lt_unit_make(s_share, groups, s_nact, s_total1, s_split, i, sh.d, pl.n1);
    };
    auto umeta_at = [&](int i) -> uint32_t { return i < kTcMaxUnits ? s_umeta[i] : lt_unit_meta(unit_at(i)); };

    if (!go) {
        // the grid-wide meeting gave up (reported): nothing is started
    } else if (warp == 0) {
        const uint64_t wpolicy = l2_evict_first_policy();
        // ------------------------------------------------------------------ TMA producer
        if (Q4 && lane == 0) {
            // int4: two cursors over the same sequence of stages.  The packed tiles and scales go
            // into the stage ring (a slot is free once the dequantising warps have read it); the
            // token tiles go into the slot of the dequantised-tile ring they are used with (free
            // once the MMAs that read it have completed; their bytes are counted by the barrier
            // the dequantising warps arrive on, so that an MMA issuer waits once), and in the
            // second projection only when their wave's activations are written.  One thread
            // serves both, so it polls.
            constexpr int KG = kTcQ4KG;
            const int n_routed = p.B * sh.k;
            int pi = 0, ti = 0;                          // unit of each cursor
            TcUnit pu{}, tu{};
            bool pu_ok = false, tu_ok = false;           // the cursor's unit has been read from the table
            int pkt = 0, tkt = 0;
            int s = 0, ta = 0;
            uint32_t ring_par = 1, t_par = 1;
            int ready_w = 0;
            unsigned idle = 0;
            bool alive = true;
            if (Q4) asm volatile("fence.proxy.async.global;" ::: "memory");   // the permuted hidden states were written by ordinary stores

            while (alive) {
                if (!(pu_ok && tu_ok)) {
                    // (rare) a cursor stands at the end of what it has read of the table
                    if (!pu_ok && pi < n_known) { pu = unit_at(pi); pkt = pu.kt0; pu_ok = true; }
                    if (!tu_ok && ti < n_known) { tu = unit_at(ti); tkt = tu.kt0; tu_ok = true; }
                    if (!pu_ok && !tu_ok) {
                        // both at the end of what is decoded: more of the table, or the end
                        const int m = more_units(pi);
                        if (m < 0) { atomicExch(ws.status, ST_DEP_TIMEOUT); break; }
                        if (m == 0) break;
                        continue;
                    }
                }
                bool progress = false;
                if (pu_ok && mbar_test(&empty_bar[s], ring_par)) {

                    const TcGroup &g = groups[pu.a];
                    const bool shared = g.group >= sh.E;
                    const int e = shared ? g.group - sh.E : g.group;
                    const int row0 = e * (pu.mat == 2 ? sh.d : g.f) + pu.rb * 128;
                    // packed k-tiles (32 bytes of every row each) and the 8 scales per row of the 256
                    // columns they lie in (x in scales; kt0 is a multiple of 4)
                    const int mi = (shared ? 3 : 0) + pu.mat;
                    const CUtensorMap *pm = &maps.m[KG == 1 ? mi : (KG == 2 ? 15 + mi : 21 + mi)];
                    uint8_t *stage = ring + (size_t)s * pl.stage_bytes;
                    mbar_expect_tx(&full_bar[s], KG * kTcQ4Packed + kTcQ4Scales);
                    tma_load_2d_stream(stage, pm, pkt * 32, row0, &full_bar[s], wpolicy);
                    tma_load_2d(stage + KG * kTcQ4Packed, &maps.m[9 + mi], (pkt & ~3) * 2, row0, &full_bar[s]);
                    tc_ring_next(s, ring_par, S);
                    pkt += KG;
                    if (pkt >= pu.kt1) {
                        if (++pi < n_known) { pu = unit_at(pi); pkt = pu.kt0; }
                        else pu_ok = false;
                    }
                    progress = true;

                }
                if (tu_ok) {
                    const int wv = tu.wave;
                    bool ready = tu.phase == 1 || wv < ready_w;
                    if (!ready && s_ready[wv]) {
                        // the activations of this wave are written: order them before the copies below
                        __threadfence_block();
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                        ready_w = wv + 1;
                        ready = true;
                    }
                    if (ready && mbar_test(&a_empty[ta], t_par)) {

                        uint8_t *op = tokring + (size_t)ta * KG * pl.tokb;
                        if (tu.phase == 1) {
                            // the hidden-state tiles of all KG k-tiles in one copy: [k-tile][tokb / 128 rows]
                            mbar_expect_tx(&a_full[ta], (uint32_t)(KG * pl.tokb));
                            tma_load_3d(op, &maps.m[6], 0, 0, tkt, &a_full[ta]);
                        } else {
                            // one copy per 8 slots for all KG k-tiles: [hi | lo][k-tile][8 rows]
                            const TcGroup &g = groups[tu.a];
                            const bool shared = g.group >= sh.E;
                            const int srow = shared ? g.off - n_routed : g.off;
                            mbar_expect_tx(&a_full[ta], (uint32_t)(KG * tu.n * 128));
                            for (int r = 0; r < tu.n / 2; r += 8)
                                tma_load_4d(op + r * 256 * KG, &maps.m[shared ? 8 : 7], 0, srow + r, tkt, 0, &a_full[ta]);
                        }
                        tc_ring_next(ta, t_par, pl.a_stages);
                        tkt += KG;
                        if (tkt >= tu.kt1) {
                            if (++ti < n_known) { tu = unit_at(ti); tkt = tu.kt0; }
                            else tu_ok = false;
                        }
                        progress = true;

                    }
                }
                if (progress) {
                    idle = 0;
                } else {
                    // nothing to issue: leave the scheduler to the dequantising warps for a while
                    __nanosleep(100);
                    if (++idle > kTcSpinLimit) {
                        atomicExch(ws.status, ST_MBAR_TIMEOUT);
                        alive = false;
                    }
                }
            }

        } else if (lane == 0) {
            unsigned it = 0;
            bool alive = true;
            int ready_w = 0;
            // phase-2 stages whose weight tile is in flight but whose token tiles wait for the
            // activations (second grid-wide counter)
            int pend_wave = 0;
            int pend_n = 0, pend_stage[kTcMaxStages], pend_kt[kTcMaxStages], pend_row[kTcMaxStages], pend_shared[kTcMaxStages],
                pend_tn[kTcMaxStages];

            auto load_tokens2 = [&](int s, int kt, int srow, int shared, int tn) {
                const CUtensorMap *am = &maps.m[shared ? 8 : 7];
                uint8_t *op = ring + (size_t)s * pl.stage_bytes + pl.tok_off;
                // one copy per 8 slots: their hi rows (1 KiB) and, right behind them, their lo rows
                for (int r = 0; r < tn / 2; r += 8) tma_load_3d(op + r * 256, am, kt * 64, srow + r, 0, &full_bar[s]);
            };
            auto wait_ready = [&](int w) -> bool {

                bool ok = false;
                for (unsigned i = 0; i < kTcSpinLimit; ++i) {
                    if (s_ready[w]) { ok = true; break; }
                    __nanosleep(32);
                }

                if (!ok) { atomicExch(ws.status, ST_DEP_TIMEOUT); return false; }
                __threadfence_block();
                asm volatile("fence.proxy.async.global;" ::: "memory");
                for (int i = 0; i < pend_n; ++i) load_tokens2(pend_stage[i], pend_kt[i], pend_row[i], pend_shared[i], pend_tn[i]);
                pend_n = 0;
                ready_w = w + 1;
                return true;
            };
            const int n_routed = p.B * sh.k;
            int s = 0;                                   // ring slot of the next k-tile
            uint32_t ring_par = 1;                       // parity to wait for on its empty barrier

            for (int i = 0; alive; ++i) {
                const int m = more_units(i);
                if (m <= 0) {
                    if (m < 0) { atomicExch(ws.status, ST_DEP_TIMEOUT); alive = false; }
                    break;
                }
                const TcUnit t = unit_at(i);
                const TcGroup &g = groups[t.a];
                const bool shared = g.group >= sh.E;
                const int e = shared ? g.group - sh.E : g.group;
                const CUtensorMap *wmap = &maps.m[(shared ? 3 : 0) + t.mat];
                const int rows_per_e = t.mat == 2 ? sh.d : g.f;
                const int row0 = e * rows_per_e + t.rb * 128;
                const int srow = shared ? g.off - n_routed : g.off;   // row in the routed / shared activation array
                const int wv = t.wave;
                bool ready = t.phase == 1 || wv < ready_w;
                if (!ready) {
                    // the pending tiles all belong to one wave (pend_wave); if that is an earlier wave than
                    // this unit's, it has to become ready before tiles of this wave may be pending.  (A CTA
                    // without second-projection units of wave 0 reaches here with ready_w still 0 and
                    // tiles of wave 1 pending: those must wait for wave 1, not for wave 0.)
                    if (pend_n > 0 && wv > pend_wave) { if (!wait_ready(pend_wave)) { alive = false; break; } }
                    if (s_ready[wv]) {
                        alive = wait_ready(wv);
                        ready = alive;
                    }
                }

                for (int kt = t.kt0; kt < t.kt1 && alive; ++kt, ++it, tc_ring_next(s, ring_par, S)) {
                    if (!ready && pend_n == S) {
                        if (!wait_ready(wv)) { alive = false; break; }     // every slot waits for tokens
                        ready = true;
                    }

                    if (!mbar_wait(&empty_bar[s], ring_par)) {
                        atomicExch(ws.status, ST_MBAR_TIMEOUT);
                        alive = false;
                        break;
                    }

                    uint8_t *stage = ring + (size_t)s * pl.stage_bytes;
                    const uint32_t op_bytes = t.phase == 1 ? (pl.x_bytes ? 0u : (uint32_t)t.n * 128u) : (uint32_t)t.n * 128u;
                    mbar_expect_tx(&full_bar[s], kTcWTile + op_bytes);
                    tma_load_2d_stream(stage, wmap, kt * 64, row0, &full_bar[s], wpolicy);
                    if (t.phase == 1) {
                        if (!pl.x_bytes)
                            for (int r = 0; r < t.n; r += 16)
                                tma_load_2d(stage + pl.tok_off + r * 128, &maps.m[6], kt * 64, r, &full_bar[s]);
                    } else if (ready) {
                        load_tokens2(s, kt, srow, shared, t.n);
                    } else {
                        pend_stage[pend_n] = s; pend_kt[pend_n] = kt; pend_row[pend_n] = srow;
                        pend_shared[pend_n] = shared; pend_tn[pend_n] = t.n;
                        pend_wave = wv;
                        ++pend_n;
                    }

                }
            }
            if (alive && pend_n > 0) wait_ready(pend_wave);

        }
    } else if (warp == 1 || warp == 6 || (Q4 && warp >= 11 + kTcQ4DeqWarps)) {
        // ------------------------------------------------------------------ MMA issuers
        // Issuing one tcgen05 instruction (an MMA or a commit) costs a thread on the order of 150
        // cycles whatever its shape, and with N = 16 every MMA covers only 4 KiB of weights, so
        // several warps share the work: with two issuers, issuer h takes K-steps 2h and 2h + 1 of
        // every k-tile, with four (int4 path) K-step h; each accumulates into its own TMEM columns
        // and the epilogue adds the partial accumulators.
        const int half = warp == 1 ? 0 : (warp == 6 ? 1 : warp - (9 + kTcQ4DeqWarps));     // with one issuer (int4, many tokens): warp 1
        if (lane == 0 && half < NI) {
            unsigned it = 0, ui = 0;
            int buf = 0;                                 // accumulator buffer of the current run, and the parity
            uint32_t buf_par = 1;                        // to wait for on its "drained" barrier
            uint32_t acc = 0;
            bool alive = true;
            int s = 0;
            uint32_t ring_par = 0;
            int ta = 0;                                  // int4: slot and parity of the dequantised-tile ring
            uint32_t a_par = 0;
            if (pl.x_bytes && half == 0) {
                // all token tiles of the hidden states, once (this thread has nothing to issue before they land)
                mbar_expect_tx(&x_bar, (uint32_t)pl.x_bytes);
                for (int kt = 0; kt < (sh.d + 63) / 64; ++kt)
                    for (int r = 0; r < pl.n1; r += 16)
                        tma_load_2d(xres + ((size_t)kt * pl.n1 + r) * 128, &maps.m[6], kt * 64, r, &x_bar);
            }
            if (pl.x_bytes && !mbar_wait(&x_bar, 0)) {
                atomicExch(ws.status, ST_MBAR_TIMEOUT);
                alive = false;
            }
            // descriptor halves (see tc_mma_bf16_parts); K-step k of a 64-wide tile lies 32 bytes further
            const uint32_t ks = 4u / (uint32_t)NI, koff = 2u * ks * (uint32_t)half;
            const uint32_t hi_std = (uint32_t)(tc_smem_desc(ring) >> 32);
            const uint32_t hi_p2 = Q4 ? (uint32_t)(tc_smem_desc_sbo(ring, (uint32_t)kTcQ4KG * 1024u) >> 32) : hi_std;
            const uint32_t ring_lo = (uint32_t)tc_smem_desc(ring) + koff, xres_lo = (uint32_t)tc_smem_desc(xres) + koff;
            const uint32_t tok_lo = (uint32_t)tc_smem_desc(tokring) + koff;
            const uint32_t a_tmem0 = tmem_base + (uint32_t)kTcQ4ACol + 4u * koff;     // 8 columns per K-step

            if (Q4) {
                // int4: a unit is one stage; everything this thread needs of it is one word
                uint32_t d_tmem = tmem_base + (uint32_t)(half * 2 * pl.n1), buf = 0, run_par = 1;
                const uint32_t tok_slot = (uint32_t)kTcQ4KG * ((uint32_t)pl.tokb >> 4), tok_step1 = (uint32_t)pl.tokb >> 4;
                for (;; ++ui) {
                    const int m = more_units((int)ui);
                    if (m <= 0) {
                        if (m < 0) atomicExch(ws.status, ST_DEP_TIMEOUT);
                        break;
                    }
                    const uint32_t um = umeta_at((int)ui);
                    if (um & 1u) {

                        if (!mbar_wait(&acc_empty[buf], run_par)) { atomicExch(ws.status, ST_MBAR_TIMEOUT); break; }

                        acc = 0;
                    }

                    // the unit as bf16 in tensor memory, written by the dequantising warps, and its token tiles
                    if (!mbar_wait(&a_full[ta], a_par)) { atomicExch(ws.status, ST_MBAR_TIMEOUT); break; }

                    tc_fence_after();
                    {
                        // dequantised k-tiles of slot ta (32 columns each) and their token tiles: phase 1
                        // [k-tile][rows], phase 2 [8 slots][hi | lo][k-tile][8 rows] (8-row groups KG KiB apart)
                        const uint32_t idesc = tc_idesc_f16((int)(um >> 8));
                        const bool p2 = (um & 4u) != 0;
                        uint32_t a_tm = a_tmem0 + (uint32_t)ta * (kTcQ4KG * 32u);
                        uint32_t b_lo = tok_lo + (uint32_t)ta * tok_slot;
                        const uint32_t b_step = p2 ? 64u : tok_step1, b_hi = p2 ? hi_p2 : hi_std;
#pragma unroll
                        for (int g = 0; g < kTcQ4KG; ++g, a_tm += 32u, b_lo += b_step) {
                            for (uint32_t k = 0; k < ks; ++k) {
                                tc_mma_bf16_tmem_a(d_tmem, a_tm + 8 * k, b_lo + 2 * k, b_hi, idesc, acc);
                                acc = 1;
                            }
                        }
                    }
                    tc_commit(&a_empty[ta]);           // frees the dequantised tiles and the token tiles
                    tc_ring_next(ta, a_par, pl.a_stages);
                    if (um & 2u) {
                        tc_commit(&acc_full[buf]);
                        buf ^= 1u;
                        if (buf == 0) run_par ^= 1u;
                        d_tmem = tmem_base + (uint32_t)(buf * 2 * NI * pl.n1 + half * 2 * pl.n1);
                    }

                }
            } else
            for (; alive; ++ui) {
                const int m = more_units((int)ui);
                if (m <= 0) {
                    if (m < 0) atomicExch(ws.status, ST_DEP_TIMEOUT);
                    break;
                }
                const TcUnit t = unit_at((int)ui);
                if (t.first) {

                    if (!mbar_wait(&acc_empty[buf], buf_par)) {
                        atomicExch(ws.status, ST_MBAR_TIMEOUT);
                        break;
                    }

                    tc_fence_after();
                    acc = 0;
                }
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 2 * NI * pl.n1 + half * 2 * pl.n1);
                // phase 2: every 16 columns are the hi rows and the lo rows of 8 slots; the epilogue
                // adds the two halves
                const uint32_t idesc = tc_idesc(t.n);
                for (int kt = t.kt0; kt < t.kt1; ++kt, ++it, tc_ring_next(s, ring_par, S)) {

                    if (!mbar_wait(&full_bar[s], ring_par)) {
                        atomicExch(ws.status, ST_MBAR_TIMEOUT);
                        alive = false;
                        break;
                    }

                    tc_fence_after();

                    {
                        const uint32_t a_lo = ring_lo + (uint32_t)s * ((uint32_t)pl.stage_bytes >> 4);
                        const uint32_t b_lo = (t.phase == 1 && pl.x_bytes) ? xres_lo + (uint32_t)kt * ((uint32_t)pl.n1 * 8u)
                                                                           : a_lo + ((uint32_t)pl.tok_off >> 4);
                        for (uint32_t k = 0; k < ks; ++k) {       // K = 16 steps inside the 64-wide tile: +32 bytes each
                            tc_mma_bf16_parts(d_tmem, a_lo + 2 * k, hi_std, b_lo + 2 * k, hi_std, idesc, acc);
                            acc = 1;
                        }
                    }

                    tc_commit(&empty_bar[s]);          // frees the stage when these MMAs have read it

                }
                if (alive && t.last) {
                    tc_commit(&acc_full[buf]);
                    if (++buf == NACC) { buf = 0; buf_par ^= 1u; }
                }
            }

        }
    } else if (Q4 && warp >= 11) {
        // ------------------------------------------------------------------ dequantising warps (int4)
        // Every row of a packed k-tile (64 nibbles, stored q + 8) becomes 64 binary16 values
        // q * scale, written to tensor memory as the A operand of the MMAs (row = lane, two values
        // per 32-bit column): per 32-bit word eight nibbles -> 1024 + n or 1024 + 16 n as binary16
        // by an OR into the mantissa, then n - 8 (exact), times the block's scale (binary16 as
        // stored, so the product is the only rounding: 2^-12 relative).  Scales that lie past the
        // matrix read as 0 (TMA fill), so a ragged last tile contributes nothing.
        // A stage holds KG k-tiles: per row 2 * KG chunks of 16 packed bytes (32 weights, one
        // scale each).  A warp reaches the 32 lanes of its quarter (warp index mod 4) only, so
        // thread (r, h) takes row r = 32 * (warp mod 4) + lane and chunks h * KG .. h * KG + KG - 1,
        // h = 0 for the first four warps, 1 for the others.
        const int r = 32 * (warp & 3) + lane, h = (warp - 11) >> 2;
        constexpr int KG = kTcQ4KG;
        constexpr int CP = 2 * KG / (kTcQ4DeqWarps / 4);      // chunks of its row per thread
        int s = 0, ta = 0;
        uint32_t ring_par = 0, a_par = 1;
        bool alive = true;
        const __half2 minus1032 = __floats2half2_rn(-1032.0f, -1032.0f), sixteenth = __floats2half2_rn(0.0625f, 0.0625f),
                      minus72 = __floats2half2_rn(-72.0f, -72.0f);
        const uint32_t a_lane = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)kTcQ4ACol;

        // contraction lengths are multiples of 256 here, so every unit is exactly one stage and
        // nothing of it has to be decoded
        {
            for (int ui = 0; alive; ++ui, tc_ring_next(s, ring_par, S), tc_ring_next(ta, a_par, pl.a_stages)) {
                const int m = more_units(ui);
                if (m <= 0) {
                    if (m < 0 && lane == 0) atomicExch(ws.status, ST_DEP_TIMEOUT);
                    break;
                }

                const bool ok_full = mbar_wait(&full_bar[s], ring_par);

                if (!ok_full || !mbar_wait(&a_empty[ta], a_par)) {
                    if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                    alive = false;
                    break;
                }
                tc_fence_after();                  // the MMAs that read this slot have completed

                const uint8_t *stage = ring + (size_t)s * pl.stage_bytes;
                const uint8_t *prow = stage + (size_t)r * (32 * KG);
                uint32_t sc[2];                    // this thread's CP scales (binary16) in one load
                if (CP == 4) {
                    const uint2 v = *reinterpret_cast<const uint2 *>(stage + KG * kTcQ4Packed + r * 16 + h * 8);
                    sc[0] = v.x; sc[1] = v.y;
                } else {
                    sc[0] = *reinterpret_cast<const uint32_t *>(stage + KG * kTcQ4Packed + r * 16 + h * 4); sc[1] = 0;
                }
                const uint32_t a_slot = a_lane + (uint32_t)(ta * KG) * 32u;
#pragma unroll
                for (int qi = 0; qi < CP; ++qi) {
                    const int q = h * CP + qi;                         // chunk of 32 weights inside the stage
                    // the packed rows are swizzled over their own width by the TMA copy
                    const int sw = KG == 4 ? (r & 7) : (KG == 2 ? ((r >> 1) & 3) : ((r >> 2) & 1));
                    const uint4 pk = *reinterpret_cast<const uint4 *>(prow + ((q ^ sw) * 16));
                    // the block's scale is binary16 already: both halves of a register
                    const uint32_t sc2u = __byte_perm(sc[qi >> 1], 0u, (qi & 1) ? 0x3232u : 0x1010u);
                    const __half2 sc2 = *reinterpret_cast<const __half2 *>(&sc2u);
                    const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
                    uint32_t o[16];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        // A nibble n OR-ed into the mantissa of binary16 1024 is 1024 + n exactly; one
                        // that sits four bits higher gives 1024 + 16 n, which one fused multiply-add
                        // (x / 16 - 72) turns into the same n - 8 without a shift.  So a 32-bit word
                        // costs one shift and four logic instructions, and the pairs come out as
                        // (n0, n4), (n1, n5), (n2, n6), (n3, n7): the token tiles carry the same
                        // permutation of every 8 columns, so no instruction is spent on reordering.
                        // n - 8 is exact; the product with the scale rounds once (2^-12 relative).
                        const uint32_t mlo = 0x000F000Fu, mhi = 0x00F000F0u, k1024 = 0x64006400u;
                        const uint32_t w8 = w[c] >> 8;
                        uint32_t e[4];
                        tc_nibble_pair(e[0], w[c], mlo, k1024);
                        tc_nibble_pair(e[1], w[c], mhi, k1024);
                        tc_nibble_pair(e[2], w8, mlo, k1024);
                        tc_nibble_pair(e[3], w8, mhi, k1024);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const __half2 x = *reinterpret_cast<const __half2 *>(&e[j]);
                            const __half2 qv = (j & 1) ? __hfma2(x, sixteenth, minus72) : __hadd2(x, minus1032);
                            const __half2 v = __hmul2(qv, sc2);
                            o[4 * c + j] = *reinterpret_cast<const uint32_t *>(&v);
                        }
                    }
                    tc_st16(a_slot + (uint32_t)q * 16u, o);          // k-tile q / 2, its columns 16 * (q % 2) ..
                }

                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&a_full[ta]);
                    mbar_arrive(&empty_bar[s]);        // the packed tiles have been read
                }

            }
        }

    } else if (warp == 10) {
        // ------------------------------------------------------------------ watcher
        // polls the waves' second counters (all CTAs have written their slice of the activations)
        // and publishes them in shared memory, so that the producer never waits on global memory
        if (lane == 0) {
            const int W = s_split < s_nact ? 2 : 1;
            for (int w = 0; w < W; ++w) {
                bool ok = false;
                for (unsigned i = 0; i < (1u << 21); ++i) {
                    if (ld_acquire(&ws.sync[kTcReady - 4 + w]) >= (int)gridDim.x) { ok = true; break; }
                    __nanosleep(32);
                }
                if (!ok) { atomicExch(ws.status, ST_DEP_TIMEOUT); break; }
                __threadfence_block();
                s_ready[w] = 1;

            }
        }
    } else if (warp >= 7) {
        // ------------------------------------------------------------------ converter warps
        // per wave: wait for this CTA's hand-over, arrive on the wave's grid-wide counter, wait
        // (bounded) for all CTAs, convert this CTA's slice of the wave, arrive on the second counter
        const int et = tid - 224;                      // 0..95 among the converter threads
        const int n_routed = p.B * sh.k;
        uint32_t ep_phase = 0;                         // running parity of cv_bar
        uint64_t *ep_bar_p = &cv_bar;
        const long long n_el = (long long)n_routed * sh.f + (long long)sh.n_sh * p.B * sh.f_sh;
        const int n_active = s_nact, a_split = s_split, W = a_split < n_active ? 2 : 1;

        auto wave_convert = [&](int w) -> bool {

            if (et == 0) {
                bool ok = false;
                for (unsigned i = 0; i < (kTcSpinLimit >> 2); ++i) {
                    if (ld_acquire(&ws.sync[kTcReady - 8 + w]) >= (int)gridDim.x) { ok = true; break; }
                    __nanosleep(16);
                }
                if (!ok) atomicExch(ws.status, ST_DEP_TIMEOUT);
                s_flag = ok;

            }
            if (!tc_bar(ep_bar_p, ep_phase, lane)) return false;
            if (!s_flag) return false;
            __threadfence_block();                 // the counter was read with acquire by one thread of this barrier

            // pre holds a gate plane and an up plane, both indexed exactly like the activations
            // (act_offset(slot) + row).  The wave's groups, one behind the other in group order, form
            // one range of elements; this CTA converts a contiguous slice of it, four elements per
            // thread and step (a group's elements are contiguous, the groups of a wave need not be)
            const int g_lo = w == 0 ? 0 : a_split, g_hi = (w == 0 && W == 2) ? a_split : n_active;
            const long long base = s_epfx[g_lo], n4 = ((long long)s_epfx[g_hi] - base) >> 2;
            const long long lo4 = n4 * blockIdx.x / gridDim.x, hi4 = n4 * (blockIdx.x + 1) / gridDim.x;
            for (int a = g_lo; a < g_hi; ++a) {
            const long long ga4 = ((long long)s_epfx[a] - base) >> 2, gb4 = ((long long)s_epfx[a + 1] - base) >> 2;
            const long long qa = lo4 > ga4 ? lo4 : ga4, qb = hi4 < gb4 ? hi4 : gb4;
            const long long abs0 = (long long)act_offset(groups[a].off, n_routed, sh.f, sh.f_sh) - 4 * ga4;
            for (long long q = qa + et; q < qb; q += 96) {
                const long long i = abs0 + 4 * q;
                const float4 gv = __ldcg(reinterpret_cast<const float4 *>(p.pre + i));
                const float4 uv = __ldcg(reinterpret_cast<const float4 *>(p.pre + n_el + i));
                const float a0 = silu_mul(gv.x, uv.x), a1 = silu_mul(gv.y, uv.y), a2 = silu_mul(gv.z, uv.z),
                            a3 = silu_mul(gv.w, uv.w);
                if (Q4) {
                    // binary16 hi + lo parts (the int4 path's operand format).  Columns i .. i + 3 of
                    // their group of 8 go to positions 0, 2, 4, 6 (first half of the group) or
                    // 1, 3, 5, 7 (second half): the order the dequantised weights are in
                    const __half2 h01 = __floats2half2_rn(a0, a1), h23 = __floats2half2_rn(a2, a3);
                    const __half2 l01 = __floats2half2_rn(a0 - __low2float(h01), a1 - __high2float(h01));
                    const __half2 l23 = __floats2half2_rn(a2 - __low2float(h23), a3 - __high2float(h23));
                    const long long g8 = i & ~7ll;
                    const int odd = (int)((i >> 2) & 1);
                    __half *ph = reinterpret_cast<__half *>(p.act_hi) + g8 + odd, *pq = reinterpret_cast<__half *>(p.act_lo) + g8 + odd;
                    ph[0] = __low2half(h01); ph[2] = __high2half(h01); ph[4] = __low2half(h23); ph[6] = __high2half(h23);
                    pq[0] = __low2half(l01); pq[2] = __high2half(l01); pq[4] = __low2half(l23); pq[6] = __high2half(l23);
                } else {
                    const __nv_bfloat162 h01 = __floats2bfloat162_rn(a0, a1), h23 = __floats2bfloat162_rn(a2, a3);
                    const __nv_bfloat162 l01 = __floats2bfloat162_rn(a0 - __low2float(h01), a1 - __high2float(h01));
                    const __nv_bfloat162 l23 = __floats2bfloat162_rn(a2 - __low2float(h23), a3 - __high2float(h23));
                    uint2 hv, lv;
                    hv.x = *reinterpret_cast<const uint32_t *>(&h01); hv.y = *reinterpret_cast<const uint32_t *>(&h23);
                    lv.x = *reinterpret_cast<const uint32_t *>(&l01); lv.y = *reinterpret_cast<const uint32_t *>(&l23);
                    *reinterpret_cast<uint2 *>(p.act_hi + i) = hv;
                    *reinterpret_cast<uint2 *>(p.act_lo + i) = lv;
                }
            }
            }
            // the activations are read by TMA copies of other CTAs: proxy fence over global memory by
            // every writer, then one release at GPU scope behind the barrier of the converter warps
            asm volatile("fence.proxy.async.global;" ::: "memory");
            if (!tc_bar(ep_bar_p, ep_phase, lane)) return false;
            if (et == 0) { tc_red_release(&ws.sync[kTcReady - 4 + w]);  }

            return true;
        };

        for (int w = 0; w < W; ++w) {
            // the hand-over may come late in the kernel: a long but bounded wait
            bool ok = false;
            for (unsigned i = 0; i < (1u << 22); ++i) {
                if (mbar_try_wait(&conv_go[w], 0)) { ok = true; break; }
                __nanosleep(24);
            }
            if (!ok) { if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT); break; }
            if (et == 0) tc_red_release(&ws.sync[kTcReady - 8 + w]);   // orders the CTA's reductions, observed through conv_go
            if (!wave_convert(w)) break;
        }

    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;                        // TMEM lane quarter this warp may read
        const int et = tid - 64;                       // 0..127 among the epilogue threads
        unsigned ui = 0;
        int buf = 0;                                   // accumulator buffer of the next run to drain, and the parity
        uint32_t buf_par = 0;                          // to wait for on its "complete" barrier
        const int n_routed = p.B * sh.k;
        bool alive = true;

        // ---- hand-over between the projections, per wave (see the header comment)
        const int n_routed_el = n_routed;   // (alias used below)
        (void)n_routed_el;
        const long long n_el = (long long)n_routed * sh.f + (long long)sh.n_sh * p.B * sh.f_sh;
        const int n_units = s_nunits[2], W = s_split < s_nact ? 2 : 1;
        const int a_split = s_split;
        // (where the CTA's sequence stands in front of a unit: 0 in wave 0's first projection, 1 in
        // wave 1's, 2 behind both: second projection, or the end)
        int next_arrive = 0;
        auto wave_arrive = [&](int w) -> bool {
            // this CTA's phase-1 reductions of wave w are issued: hand over to the converter warps,
            // whose first thread orders them (fence) before it arrives on the grid-wide counter, so
            // that no epilogue thread stalls on a fence
            __syncwarp();
            if (lane == 0) mbar_arrive(&conv_go[w]);
            return true;
        };
        // called before every unit (and once at the end): hand a wave over once this CTA's phase-1
        // units of it are all done
        auto service = [&](int stage) -> bool {
            while (next_arrive < W && stage > next_arrive) {
                if (!wave_arrive(next_arrive)) return false;
                ++next_arrive;
            }
            return true;
        };
        {
            for (; (int)ui < n_units && alive; ++ui) {
                const TcUnit t = unit_at((int)ui);
                if (!service(t.phase == 2 ? 2 : (t.a >= a_split ? 1 : 0))) { alive = false; break; }
                if (!t.last) continue;                 // the run's accumulator is read after its last unit
                const TcGroup &g = groups[t.a];

                if (!mbar_wait(&acc_full[buf], buf_par)) {
                    if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                    alive = false;
                    break;
                }

                tc_fence_after();
                {
                const int row = t.rb * 128 + q * 32 + lane;           // row of the matrix inside the expert
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 2 * NI * pl.n1);
                const uint32_t other = (uint32_t)(2 * pl.n1);      // the next issuer's partial accumulator
                if (t.phase == 1) {
                    const bool row_ok = row < g.f;
                    // slot of the expert's i-th token = g.off + i; walk its tokens in ascending order
                    float *dst = p.pre + (size_t)t.mat * n_el + act_offset(g.off, n_routed, sh.f, sh.f_sh) + row;
                    const size_t slot_stride = (size_t)g.f;
                    for (int c = 0; c < t.n; c += 16) {
                        float v[16], v2[16];
                        tc_ld16(taddr + c, v);
                        for (int h = 1; h < NI; ++h) {
                            tc_ld16(taddr + h * other + c, v2);
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] += v2[i];
                        }
                        const unsigned m16 = (unsigned)((g.mask >> c) & 0xffffull);
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            if (((m16 >> i) & 1u) && row_ok) {
                                const int rank = __popcll(g.mask & ((1ull << (c + i)) - 1ull));
                                atomicAdd(dst + rank * slot_stride, v[i]);
                            }
                        }
                    }
                } else {
                    const bool row_ok = row < sh.d;
                    for (int c = 0; c < t.n; c += 16) {
                        float v[16], v2[16];                      // columns: 8 hi, 8 lo of slots c / 2 .. c / 2 + 7
                        tc_ld16(taddr + c, v);
                        for (int h = 1; h < NI; ++h) {
                            tc_ld16(taddr + h * other + c, v2);
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] += v2[i];
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int ti = (c >> 1) + i;
                            if (ti < g.T && row_ok) {
                                const int slot = g.off + ti;
                                atomicAdd(&p.y[(size_t)s_slot_token[slot] * sh.d + row],
                                          s_slot_w[slot] * (v[i] + v[i + 8]));
                            }
                        }
                    }
                }
                }
                // the accumulator may be overwritten
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[buf]);
                if (++buf == NACC) { buf = 0; buf_par ^= 1u; }

            }
            if (alive && !service(2)) alive = false;
        }

    }
    // every path ends here (all waits above are bounded), so the TMEM is always returned
    tc_fence_before();
    __syncthreads();

    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)pl.tmem_cols)
                     : "memory");
    }
}

}  // namespace fused
}  // namespace s2moe
