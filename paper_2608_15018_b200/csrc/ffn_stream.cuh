// Streaming expert kernel (kernel plan 2): one persistent CTA per SM reads every
// selected expert's weights from HBM exactly once through a ring of TMA bulk copies
// and contracts them with the draft tokens on the tensor cores.
//
// Work items are "stages": the bytes one consumer warp turns into finished outputs.
//   phase 1 stage: 4 gate rows + 4 up rows of one expert, all of K = d (two contiguous
//                  copies).  The hidden states of ALL B tokens stay resident in shared
//                  memory, the contraction runs over all of them, and only the tokens
//                  bucketed to this expert store a = silu(g) * u (as bf16 hi + lo).
//   phase 2 stage: 8 down rows of one expert over one K-slice of f, contracted with
//                  the expert's activations (resident operand), y += p * result.
// Phase-1 stages are dealt round-robin to the CTAs; phase-2 stages are split into one
// contiguous range per CTA so that a CTA needs the activations of one or two experts
// only.  A phase-2 operand load waits on a counter of that expert's finished phase-1
// stages.  Every wait in the kernel is bounded and reports through the status word.
//
// Inside a CTA one producer warp issues the copies; every ring slot belongs to one consumer
// warp, which finishes the stages landing there alone (no CTA-wide barrier anywhere).
// The contraction is mma.sync m16n8k16 with tokens as the M operand and eight weight
// rows as the N operand.  The K index inside every 32-wide step is permuted identically
// for both operands, so each lane feeds the tensor core from one 128-bit shared-memory
// load per row; the two 4-row halves of a stage are placed 64 bytes apart modulo 128 so
// that those loads are free of bank conflicts.
#pragma once

#include "common.cuh"

namespace s2moe {

constexpr int kStConsumerWarps = 7;   // + 1 producer warp = 256 threads, so a thread may use 255 registers
constexpr int kStThreads = (kStConsumerWarps + 1) * 32;
constexpr int kStMaxStages = 8;
constexpr int kStMaxGroups = kMaxExperts + kMaxShared;
constexpr unsigned kStSpinLimit = 1u << 20;   // bounded waits: a poll takes between some tens of ns and kMbarSuspendNs, so about a second at most
constexpr int kStMaxSmem = 232448 - 2048;     // dynamic shared memory the kernel may use

// Per-call plan, computed on the host (st_make_plan) and passed by value.
struct StPlan {
    int feasible;
    int n_cta;
    int stages;       // ring slots
    int slot_bytes;   // bytes per ring slot
    int x_pitch;      // bytes per token row of the resident hidden states (d*2 + 64)
    int x_bytes;      // pad8(B) * x_pitch
    int op_cap;       // capacity of the phase-2 operand region
    int alias;        // 1: the operand region is the hidden-state region (drained first)
    int tab_bytes;    // group and slot tables
    int smem_bytes;   // total dynamic shared memory
};

struct StGroup {      // one active group, in shared memory
    unsigned long long mask;   // tokens of the batch bucketed to this group
    int group, T, off, f;      // group id, tokens, first slot, inner dim
    int p1, p2;                // first phase-1 / phase-2 stage of the group
    int nks, ksl;              // K-slices of a phase-2 row and their length
};

struct StageDesc {
    int phase, gslot, tile, ks;   // gslot: index into the active list
    int klen, op_gen, rc, pad_;   // K elements, operand generation, row chunk bytes
};

struct StreamArgs {
    Shape sh;
    LayerPtrs lp;
    Workspace ws;
    StPlan plan;
    const void *hidden;
    float *y;
    __nv_bfloat16 *act_hi, *act_lo;
    int B;
    size_t act_elems;   // elements of act_hi / act_lo
};

// ---- shapes shared by the host planner, the gating kernel and this kernel ----------

__host__ __device__ __forceinline__ int st_pad8(int t) { return (t + 7) & ~7; }

// number of K-slices of a phase-2 row of inner dim f for T tokens, given the operand
// capacity (hi and lo rows of pad8(T) tokens, each row padded by 64 bytes) and the longest
// slice a ring slot takes (kcap = d: a phase-2 stage is never larger than a phase-1 stage)
__host__ __device__ __forceinline__ int st_nks(int f, int T, int op_cap, int kcap)
{
    const int rows = 2 * st_pad8(T);
    int kmax = ((op_cap / rows - 64) / 2) & ~31;
    if (kmax > kcap) kmax = kcap & ~31;
    if (kmax < 32) kmax = 32;
    return (f + kmax - 1) / kmax;
}
__host__ __device__ __forceinline__ int st_ksl(int f, int nks) { return ((f / 32 + nks - 1) / nks) * 32; }

inline StPlan st_make_plan(const Shape &sh, int B, int n_sm, int n_slots)
{
    StPlan p{};
    const int G = sh.E + sh.n_sh;
    p.n_cta = n_sm;
    p.x_pitch = sh.d * 2 + 64;
    p.x_bytes = st_pad8(B) * p.x_pitch;
    const int fmax = sh.n_sh && sh.f_sh > sh.f ? sh.f_sh : sh.f;
    p.tab_bytes = ((int)sizeof(StGroup) * (G + 1) + 8 * n_slots + 127) & ~127;
    const int avail = kStMaxSmem - p.tab_bytes;
    const int op_full = 2 * st_pad8(B) * (fmax * 2 + 64);
    const int op_min = 2 * st_pad8(B) * (256 * 2 + 64);
    // a ring slot holds a phase-1 stage (8 rows of d) or a phase-2 stage (8 rows of one K-slice);
    // two rounds: the K-slice length depends on the operand capacity, which depends on the slot
    p.slot_bytes = 8 * sh.d * 2 + 128;
    bool fits = false;
    for (int round = 0; round < 2; ++round) {
        // one consumer warp per ring slot: as many slots (up to 7) as leave room for the whole
        // phase-2 operand next to the hidden states; at least 4, then the operand takes over the
        // hidden-state region once phase 1 has drained (alias)
        p.stages = kStConsumerWarps;
        while (p.stages > 4 && avail - p.x_bytes - p.stages * p.slot_bytes < op_full) --p.stages;
        const int left = avail - p.x_bytes - p.stages * p.slot_bytes;
        if (left >= op_full) {
            p.alias = 0;
            p.op_cap = op_full;
        } else {
            p.alias = 1;
            p.op_cap = avail - p.stages * p.slot_bytes;
            if (p.op_cap < p.x_bytes || p.op_cap < op_min) {
                p.stages = 3;
                p.op_cap = avail - p.stages * p.slot_bytes;
            }
            if (p.op_cap > op_full && op_full >= p.x_bytes) p.op_cap = op_full;
        }
        p.op_cap &= ~127;
        const int ksl_max = st_ksl(fmax, st_nks(fmax, 1, p.op_cap, sh.d));   // longest slice: fewest tokens
        const int stage2 = 8 * ksl_max * 2 + 128;
        p.smem_bytes = p.tab_bytes + (p.alias ? p.op_cap : p.x_bytes + p.op_cap) + p.stages * p.slot_bytes;
        fits = p.op_cap >= op_min && (!p.alias || p.op_cap >= p.x_bytes) && stage2 <= p.slot_bytes &&
               p.smem_bytes <= kStMaxSmem && B <= kMaxTokens;
        if (fits || stage2 <= p.slot_bytes) break;
        p.slot_bytes = stage2;
    }
    p.feasible = fits && sh.weight_dtype == DT_BF16 && sh.act_dtype == DT_BF16;
    return p;
}

// ---- PTX helpers ---------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// upper bound in nanoseconds of the time a thread may stay suspended in one try_wait (it wakes when
// the phase completes): a waiting thread then costs its scheduler next to no issue slots
constexpr uint32_t kMbarSuspendNs = 1000;
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(kMbarSuspendNs)
        : "memory");
    return ok != 0;
}
// bounded wait; false when it gave up
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity)
{
    for (unsigned i = 0; i < kStSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
#ifdef S2MOE_SELFCHECK
#define ST_BULK(ws, smem0, smem_bytes, dst, src, bytes, bar, g0, gbytes, code)                                      \
    do {                                                                                                           \
        const long long so_ = (const uint8_t *)(dst) - (const uint8_t *)(smem0);                                   \
        const long long go_ = (const uint8_t *)(src) - (const uint8_t *)(g0);                                      \
        if (st_check(ws, so_ >= 0 && so_ + (long long)(bytes) <= (long long)(smem_bytes) && (so_ & 15) == 0, (code), so_, (smem_bytes)) && \
            st_check(ws, go_ >= 0 && go_ + (long long)(bytes) <= (long long)(gbytes) && (go_ & 15) == 0 && ((bytes) & 15) == 0, (code) + 100, go_, (gbytes))) \
            bulk_g2s(dst, src, bytes, bar);                                                                        \
    } while (0)
#else
#define ST_BULK(ws, smem0, smem_bytes, dst, src, bytes, bar, g0, gbytes, code) bulk_g2s(dst, src, bytes, bar)
#endif
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <typename G>
__device__ __forceinline__ int upper_group1(const G *g, int n, int u)
{
    int lo = 0, hi = n;   // largest a with g[a].p1 <= u
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g[mid].p1 <= u) lo = mid; else hi = mid;
    }
    return lo;
}
template <typename G>
__device__ __forceinline__ int upper_group2(const G *g, int n, int u)
{
    int lo = 0, hi = n;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g[mid].p2 <= u) lo = mid; else hi = mid;
    }
    return lo;
}

// Optional self-check build (-DS2MOE_SELFCHECK): every global access and bulk copy of the
// kernel is bounds-checked; the first violation is recorded in header[8..11] as
// {code, value, limit, block} and the access is skipped.
#ifdef S2MOE_SELFCHECK
__device__ __forceinline__ bool st_check(const Workspace &ws, bool ok, int code, long long v, long long lim)
{
    if (!ok && atomicCAS(&ws.header[8], 0, code) == 0) {
        ws.header[9] = (int)v;
        ws.header[10] = (int)lim;
        ws.header[11] = (int)blockIdx.x;
        ws.header[12] = (int)(v >> 32);
    }
    return ok;
}
#define ST_CHECK(ws, cond, code, v, lim) st_check(ws, cond, code, (long long)(v), (long long)(lim))
#else
#define ST_CHECK(ws, cond, code, v, lim) true
#endif

// ---- consumer side ----------------------------------------------------------------

// One phase-1 stage: D[token][gate/up row pairs] over all of K, then SwiGLU and store.
template <int MT>
__device__ __forceinline__ void consume_phase1(const StreamArgs &p, const StGroup &grp, const StageDesc &d,
                                               const uint8_t *wreg, const uint8_t *xreg, int lane)
{
    const int g = lane >> 2, t = lane & 3;
    const int rowbytes = p.sh.d * 2;
    const uint8_t *wrow = wreg + (size_t)(g >> 1) * rowbytes + (size_t)(g & 1) * (4 * rowbytes + 64) + t * 16;
    const int bpad = st_pad8(p.B);
    float acc[MT][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[m][q] = 0.f;
    const uint8_t *xrow[MT];
    bool has1[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        xrow[m] = xreg + (size_t)(m * 16 + g) * p.plan.x_pitch + t * 16;
        has1[m] = m * 16 + g + 8 < bpad;
    }
    const size_t x8 = (size_t)8 * p.plan.x_pitch;
    const int nsteps = p.sh.d >> 5;
    // A single warp has to hide its own latencies: work in blocks of BS K-steps, load the next
    // block's operands while the current block's tensor-core instructions run, and keep
    // 2 * BS independent accumulator chains per m-tile.
    constexpr int BS = MT == 1 ? 4 : (MT == 2 ? 2 : 1);
    constexpr int NB = MT <= 2 ? 2 : 1;   // operand buffers: double-buffered while registers allow
    float ch[MT][2 * BS][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 2 * BS; ++c)
#pragma unroll
            for (int q = 0; q < 4; ++q) ch[m][c][q] = 0.f;
    uint4 w[NB][BS], xa[NB][BS][MT], xb[NB][BS][MT];
    auto load_block = [&](int buf, int s0) {
#pragma unroll
        for (int i = 0; i < BS; ++i) {
            w[buf][i] = *reinterpret_cast<const uint4 *>(wrow + (s0 + i) * 64);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                xa[buf][i][m] = *reinterpret_cast<const uint4 *>(xrow[m] + (s0 + i) * 64);
                xb[buf][i][m] = has1[m] ? *reinterpret_cast<const uint4 *>(xrow[m] + x8 + (s0 + i) * 64)
                                        : make_uint4(0, 0, 0, 0);
            }
        }
    };
    auto mma_block = [&](int buf) {
#pragma unroll
        for (int i = 0; i < BS; ++i)
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                mma_bf16(ch[m][2 * i], xa[buf][i][m].x, xb[buf][i][m].x, xa[buf][i][m].y, xb[buf][i][m].y,
                         w[buf][i].x, w[buf][i].y);
                mma_bf16(ch[m][2 * i + 1], xa[buf][i][m].z, xb[buf][i][m].z, xa[buf][i][m].w, xb[buf][i][m].w,
                         w[buf][i].z, w[buf][i].w);
            }
    };
    const int nblk = nsteps / BS;          // d is a multiple of 64, BS divides nsteps when d % 128 == 0
    if (NB == 2) {
        load_block(0, 0);
#pragma unroll 1
        for (int blk = 0; blk + 1 < nblk; blk += 2) {
            load_block(NB - 1, (blk + 1) * BS);
            mma_block(0);
            if (blk + 2 < nblk) load_block(0, (blk + 2) * BS);
            mma_block(NB - 1);
        }
        if (nblk & 1) mma_block(0);
    } else {
#pragma unroll 1
        for (int blk = 0; blk < nblk; ++blk) {
            load_block(0, blk * BS);
            mma_block(0);
        }
    }
    for (int s = nblk * BS; s < nsteps; ++s) {     // tail steps when BS does not divide nsteps
        const uint4 wv = *reinterpret_cast<const uint4 *>(wrow + s * 64);
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const uint4 va = *reinterpret_cast<const uint4 *>(xrow[m] + s * 64);
            const uint4 vb = has1[m] ? *reinterpret_cast<const uint4 *>(xrow[m] + x8 + s * 64) : make_uint4(0, 0, 0, 0);
            mma_bf16(ch[m][0], va.x, vb.x, va.y, vb.y, wv.x, wv.y);
            mma_bf16(ch[m][1], va.z, vb.z, va.w, vb.w, wv.z, wv.w);
        }
    }
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 2 * BS; ++c) sum += ch[m][c][q];
            acc[m][q] = sum;
        }
    // lane (g, t) holds (gate row t, up row t) of tokens g and g + 8 of every m-tile
    const int n_routed = p.B * p.sh.k;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int b = m * 16 + g + 8 * h;
            if (b < p.B && ((grp.mask >> b) & 1ull)) {
                const int slot = grp.off + __popcll(grp.mask & ((1ull << b) - 1ull));
                const float a = silu_mul(acc[m][2 * h], acc[m][2 * h + 1]);
                const __nv_bfloat16 hi = __float2bfloat16_rn(a);
                const __nv_bfloat16 lo = __float2bfloat16_rn(a - __bfloat162float(hi));
                const size_t o = act_offset(slot, n_routed, p.sh.f, p.sh.f_sh) + (size_t)d.tile * 4 + t;
                if (ST_CHECK(p.ws, o < p.act_elems && slot < p.ws.header[1], 1, o, p.act_elems)) {
                    p.act_hi[o] = hi;
                    p.act_lo[o] = lo;
                }
            }
        }
    }
    // release: this warp's stores, then one count for the stage
    __threadfence();
    fence_proxy_async();
    __syncwarp();
    if (lane == 0 && ST_CHECK(p.ws, d.gslot >= 0 && d.gslot < kStMaxGroups, 2, d.gslot, kStMaxGroups))
        atomicAdd(&p.ws.sync[d.gslot], 1);
}

// One phase-2 stage: D[slot][8 down rows] over one K-slice, y += p * D.
template <int MT>
__device__ __forceinline__ void consume_phase2(const StreamArgs &p, const StGroup &grp, const StageDesc &d,
                                               const uint8_t *wreg, const uint8_t *oreg, const int *slot_token,
                                               const float *slot_w, int lane)
{
    const int g = lane >> 2, t = lane & 3;
    const int rc = d.rc;                       // bytes of one weight row chunk
    const int opitch = d.klen * 2 + 64;        // operand row pitch
    const int tpad = st_pad8(grp.T);
    const uint8_t *wrow = wreg + (size_t)(g >> 1) * rc + (size_t)(g & 1) * (4 * rc + 64) + t * 16;
    float acc[MT][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[m][q] = 0.f;
    const uint8_t *hrow[MT];
    bool has1[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        hrow[m] = oreg + (size_t)(m * 16 + g) * opitch + t * 16;
        has1[m] = m * 16 + g + 8 < tpad;
    }
    const size_t o8 = (size_t)8 * opitch;
    const size_t lo_off = (size_t)tpad * opitch;
    const int nsteps = d.klen >> 5;
    // blocks of two K-steps, next block's loads in flight during the current block's
    // tensor-core instructions; four chains per step (hi / lo parts, two halves of the step)
    constexpr int BS = MT == 1 ? 2 : 1;
    constexpr int NB = MT <= 2 ? 2 : 1;
    float ch[MT][4 * BS][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 4 * BS; ++c)
#pragma unroll
            for (int q = 0; q < 4; ++q) ch[m][c][q] = 0.f;
    uint4 w[NB][BS], xa[NB][BS][MT], xb[NB][BS][MT], la[NB][BS][MT], lb[NB][BS][MT];
    auto load_block = [&](int buf, int s0) {
#pragma unroll
        for (int i = 0; i < BS; ++i) {
            const int o = (s0 + i) * 64;
            w[buf][i] = *reinterpret_cast<const uint4 *>(wrow + o);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const uint4 z = make_uint4(0, 0, 0, 0);
                xa[buf][i][m] = *reinterpret_cast<const uint4 *>(hrow[m] + o);
                la[buf][i][m] = *reinterpret_cast<const uint4 *>(hrow[m] + lo_off + o);
                xb[buf][i][m] = has1[m] ? *reinterpret_cast<const uint4 *>(hrow[m] + o8 + o) : z;
                lb[buf][i][m] = has1[m] ? *reinterpret_cast<const uint4 *>(hrow[m] + o8 + lo_off + o) : z;
            }
        }
    };
    auto mma_block = [&](int buf) {
#pragma unroll
        for (int i = 0; i < BS; ++i)
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const uint4 &A = xa[buf][i][m], &Bq = xb[buf][i][m], &L = la[buf][i][m], &M = lb[buf][i][m];
                mma_bf16(ch[m][4 * i], A.x, Bq.x, A.y, Bq.y, w[buf][i].x, w[buf][i].y);
                mma_bf16(ch[m][4 * i + 1], A.z, Bq.z, A.w, Bq.w, w[buf][i].z, w[buf][i].w);
                mma_bf16(ch[m][4 * i + 2], L.x, M.x, L.y, M.y, w[buf][i].x, w[buf][i].y);
                mma_bf16(ch[m][4 * i + 3], L.z, M.z, L.w, M.w, w[buf][i].z, w[buf][i].w);
            }
    };
    const int nblk = nsteps / BS;
    if (NB == 2) {
        if (nblk > 0) load_block(0, 0);
#pragma unroll 1
        for (int blk = 0; blk + 1 < nblk; blk += 2) {
            load_block(NB - 1, (blk + 1) * BS);
            mma_block(0);
            if (blk + 2 < nblk) load_block(0, (blk + 2) * BS);
            mma_block(NB - 1);
        }
        if (nblk & 1) mma_block(0);
    } else {
#pragma unroll 1
        for (int blk = 0; blk < nblk; ++blk) {
            load_block(0, blk * BS);
            mma_block(0);
        }
    }
    for (int s = nblk * BS; s < nsteps; ++s) {
        const int o = s * 64;
        const uint4 wv = *reinterpret_cast<const uint4 *>(wrow + o);
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const uint4 z = make_uint4(0, 0, 0, 0);
            const uint4 A = *reinterpret_cast<const uint4 *>(hrow[m] + o);
            const uint4 L = *reinterpret_cast<const uint4 *>(hrow[m] + lo_off + o);
            const uint4 Bq = has1[m] ? *reinterpret_cast<const uint4 *>(hrow[m] + o8 + o) : z;
            const uint4 M = has1[m] ? *reinterpret_cast<const uint4 *>(hrow[m] + o8 + lo_off + o) : z;
            mma_bf16(ch[m][0], A.x, Bq.x, A.y, Bq.y, wv.x, wv.y);
            mma_bf16(ch[m][1], A.z, Bq.z, A.w, Bq.w, wv.z, wv.w);
            mma_bf16(ch[m][2], L.x, M.x, L.y, M.y, wv.x, wv.y);
            mma_bf16(ch[m][3], L.z, M.z, L.w, M.w, wv.z, wv.w);
        }
    }
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 4 * BS; ++c) sum += ch[m][c][q];
            acc[m][q] = sum;
        }
    // lane (g, t): columns 2t, 2t+1 are down rows t and 4 + t of the stage
    const int r0 = d.tile * 8 + t;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int ti = m * 16 + g + 8 * h;
            if (ti < grp.T) {
                const int slot = grp.off + ti;
                const float pw = slot_w[slot];
                const size_t yo = (size_t)slot_token[slot] * p.sh.d + r0;
                float *dst = p.y + yo;
                if (ST_CHECK(p.ws, yo + 4 < (size_t)p.B * p.sh.d && slot < p.ws.header[1], 3, yo, p.B * p.sh.d)) {
                    atomicAdd(dst, pw * acc[m][2 * h]);
                    atomicAdd(dst + 4, pw * acc[m][2 * h + 1]);
                }
            }
        }
    }
}

// ---- the kernel ---------------------------------------------------------------------

__global__ void __launch_bounds__(kStThreads, 1) ffn_stream_kernel(StreamArgs p)
{
    extern __shared__ __align__(128) uint8_t st_smem[];
    __shared__ __align__(8) uint64_t full_bar[kStMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kStMaxStages];
    __shared__ __align__(8) uint64_t x_bar, op_bar;
    __shared__ StageDesc desc[kStMaxStages];

    const StPlan &pl = p.plan;
    const Shape &sh = p.sh;
    const Workspace &ws = p.ws;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_active = ws.header[0], n_slots = ws.header[1];
    const int total1 = ws.header[4], total2 = ws.header[5];
    const int G = sh.E + sh.n_sh;

    // shared memory: [group table | slot_token | slot_w | hidden states | operand | ring]
    StGroup *groups = reinterpret_cast<StGroup *>(st_smem);
    const int tab_rest = pl.tab_bytes - (int)sizeof(StGroup) * (G + 1);
    int *s_slot_token = reinterpret_cast<int *>(st_smem + sizeof(StGroup) * (G + 1));
    float *s_slot_w = reinterpret_cast<float *>(s_slot_token + tab_rest / 8);
    uint8_t *xreg = st_smem + pl.tab_bytes;
    uint8_t *oreg = pl.alias ? xreg : xreg + pl.x_bytes;
    uint8_t *ring = oreg + pl.op_cap;

    for (int a = tid; a < n_active; a += blockDim.x) {
        StGroup gr;
        gr.group = ws.active[a];
        gr.T = ws.counts[gr.group];
        gr.off = ws.offsets[gr.group];
        gr.f = gr.group < sh.E ? sh.f : sh.f_sh;
        gr.mask = ws.tokmask[gr.group];
        gr.p1 = ws.upfx1[a];
        gr.p2 = ws.upfx2[a];
        gr.nks = st_nks(gr.f, gr.T, pl.op_cap, sh.d);
        gr.ksl = st_ksl(gr.f, gr.nks);
        groups[a] = gr;
    }
    for (int i = tid; i < n_slots; i += blockDim.x) {
        s_slot_token[i] = ws.slot_token[i];
        s_slot_w[i] = ws.slot_w[i];
    }
    if (tid == 0) {
        for (int s = 0; s < pl.stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&x_bar, 1);
        mbar_init(&op_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // this CTA's work: phase-1 stages blockIdx.x, +gridDim.x, ...; phase-2 stages [lo2, hi2)
    const int P = gridDim.x;
    const int n1_mine = total1 > (int)blockIdx.x ? (total1 - 1 - (int)blockIdx.x) / P + 1 : 0;
    const int lo2 = (int)(((long long)total2 * blockIdx.x) / P);
    const int hi2 = (int)(((long long)total2 * (blockIdx.x + 1)) / P);
    const int n_mine = n1_mine + (hi2 - lo2);
    const int S = pl.stages;

    if (warp == kStConsumerWarps) {
        // ------------------------------------------------------------ producer warp
        bool alive = true;
        // hidden states of all tokens, one copy per token row
        if (lane == 0) mbar_expect_tx(&x_bar, (uint32_t)p.B * sh.d * 2);
        __syncwarp();
        for (int b = lane; b < p.B; b += 32)
            ST_BULK(ws, st_smem, pl.smem_bytes, xreg + (size_t)b * pl.x_pitch,
                    (const uint8_t *)p.hidden + (size_t)b * sh.d * 2, sh.d * 2, &x_bar, p.hidden,
                    (size_t)p.B * sh.d * 2, 10);

        int cur_a = -1, cur_ks = -1, op_gen = 0;
        for (int n = 0; n < n_mine && alive; ++n) {
            StageDesc d;
            const uint8_t *src0, *src1;   // the two 4-row halves
            const uint8_t *wbase0, *wbase1;   // tensors the halves come from (self-check build only)
            size_t rstride, wbytes = 0;
            if (n < n1_mine) {
                const int u = blockIdx.x + n * P;
                d.phase = 1;
                d.gslot = upper_group1(groups, n_active, u);
                const StGroup &gr = groups[d.gslot];
                d.tile = u - gr.p1;
                d.ks = 0;
                d.klen = sh.d;
                d.op_gen = 0;
                d.rc = sh.d * 2;
                rstride = (size_t)sh.d * 2;
                const bool shared = gr.group >= sh.E;
                const size_t e = shared ? gr.group - sh.E : gr.group;
                const size_t r0 = (e * gr.f + (size_t)d.tile * 4) * rstride;
                wbase0 = (const uint8_t *)(shared ? p.lp.sh_gate : p.lp.w_gate);
                wbase1 = (const uint8_t *)(shared ? p.lp.sh_up : p.lp.w_up);
                wbytes = (size_t)(shared ? sh.n_sh : sh.E) * gr.f * rstride;   // self-check build only
                src0 = wbase0 + r0;
                src1 = wbase1 + r0;
            } else {
                const int v = lo2 + (n - n1_mine);
                d.phase = 2;
                d.gslot = upper_group2(groups, n_active, v);
                const StGroup &gr = groups[d.gslot];
                const int local = v - gr.p2, tiles = sh.d / 8;
                d.ks = local / tiles;
                d.tile = local - d.ks * tiles;
                d.klen = min(gr.ksl, gr.f - d.ks * gr.ksl);
                d.rc = d.klen * 2;
                rstride = (size_t)gr.f * 2;
                const bool shared = gr.group >= sh.E;
                const size_t e = shared ? gr.group - sh.E : gr.group;
                wbase0 = wbase1 = (const uint8_t *)(shared ? p.lp.sh_down : p.lp.w_down);
                wbytes = (size_t)(shared ? sh.n_sh : sh.E) * sh.d * rstride;
                src0 = wbase0 + (e * sh.d + (size_t)d.tile * 8) * rstride + (size_t)d.ks * gr.ksl * 2;
                src1 = src0 + 4 * rstride;
                if (d.gslot != cur_a || d.ks != cur_ks) {
                    // new operand: (1) every stage issued so far must have been consumed (it may still
                    // read the old operand, or the hidden states the operand region aliases)
                    int ok = 1;
                    if (lane == 0) {
                        for (int back = 1; back <= S && back <= n && ok; ++back) {
                            const int m = n - back;
                            if (m < n1_mine && !pl.alias) break;   // phase-1 stages never read the operand
                            ok = mbar_wait(&empty_bar[m % S], (uint32_t)(m / S) & 1u) ? 1 : 0;
                        }
                        if (!ok) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                        // (2) every phase-1 stage of this group must have stored its activations
                        if (ok && d.gslot != cur_a) {
                            const int need = gr.f / 4;
                            ok = 0;
                            for (unsigned i = 0; i < (kStSpinLimit >> 2); ++i) {
                                if (ld_acquire(&ws.sync[d.gslot]) >= need) { ok = 1; break; }
                                __nanosleep(40);
                            }
                            if (!ok) atomicExch(ws.status, ST_DEP_TIMEOUT);
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { alive = false; break; }
                    fence_proxy_async();
                    cur_a = d.gslot;
                    cur_ks = d.ks;
                    ++op_gen;
                    const int tpad = st_pad8(gr.T), opitch = d.klen * 2 + 64;
                    if (lane == 0) mbar_expect_tx(&op_bar, (uint32_t)(2 * gr.T) * d.rc);
                    __syncwarp();
                    const size_t n_routed = (size_t)p.B * sh.k;
                    for (int r = lane; r < 2 * gr.T; r += 32) {
                        const int ti = r < gr.T ? r : r - gr.T;
                        const __nv_bfloat16 *base = r < gr.T ? p.act_hi : p.act_lo;
                        const size_t o = act_offset(gr.off + ti, (int)n_routed, sh.f, sh.f_sh) + (size_t)d.ks * gr.ksl;
                        const int srow = r < gr.T ? ti : tpad + ti;
                        ST_BULK(ws, st_smem, pl.smem_bytes, oreg + (size_t)srow * opitch, base + o, d.rc, &op_bar, base,
                                p.act_elems * 2, 20);
                    }
                }
                d.op_gen = op_gen;
            }
            const int slot = n % S;
            int ok = 1;
            if (lane == 0) ok = mbar_wait(&empty_bar[slot], (((uint32_t)(n / S)) & 1u) ^ 1u) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) {
                if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                alive = false;
                break;
            }
            uint8_t *wreg = ring + (size_t)slot * pl.slot_bytes;
            const bool contiguous = (size_t)d.rc == rstride;
            (void)wbytes; (void)wbase0; (void)wbase1;
            if (lane == 0) {
                desc[slot] = d;
                mbar_expect_tx(&full_bar[slot], (uint32_t)8 * d.rc);
            }
            __syncwarp();
            if (contiguous) {
                if (lane == 0) ST_BULK(ws, st_smem, pl.smem_bytes, wreg, src0, 4 * d.rc, &full_bar[slot], wbase0, wbytes, 30);
                if (lane == 1)
                    ST_BULK(ws, st_smem, pl.smem_bytes, wreg + 4 * d.rc + 64, src1, 4 * d.rc, &full_bar[slot], wbase1, wbytes, 40);
            } else if (lane < 8) {
                const uint8_t *src = (lane < 4 ? src0 : src1) + (size_t)(lane & 3) * rstride;
                ST_BULK(ws, st_smem, pl.smem_bytes, wreg + (size_t)(lane & 3) * d.rc + (lane < 4 ? 0 : 4 * d.rc + 64), src,
                        d.rc, &full_bar[slot], lane < 4 ? wbase0 : wbase1, wbytes, 50);
            }
        }
        if (!alive && lane == 0) {
            // let the copies that were issued land before the CTA may exit (bounded)
            for (unsigned i = 0; i < (1u << 20); ++i) __nanosleep(20);
        }
    } else {
        // ------------------------------------------------------------ consumer warps
        // Consumer warp w owns ring slot w and takes the stages n = w, w + S, ...  One waiter per
        // barrier: a parity wait is only meaningful for the phase that follows the one the
        // waiter saw complete, so two warps must never poll the same slot for different uses.
        const int mt_all = (st_pad8(p.B) + 15) >> 4;
        bool x_ready = false;
        for (int n = warp; n < n_mine && warp < S; n += S) {
            const int slot = warp;
            if (!mbar_wait(&full_bar[slot], ((uint32_t)(n / S)) & 1u)) {
                if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                break;
            }
            const StageDesc d = desc[slot];
            const StGroup &gr = groups[d.gslot];
            const uint8_t *wreg = ring + (size_t)slot * pl.slot_bytes;
            bool ok = true;
            if (d.phase == 1) {
                if (!x_ready) {
                    ok = mbar_wait(&x_bar, 0);
                    x_ready = ok;
                }
                if (ok) {
                    if (mt_all == 1) consume_phase1<1>(p, gr, d, wreg, xreg, lane);
                    else if (mt_all == 2) consume_phase1<2>(p, gr, d, wreg, xreg, lane);
                    else if (mt_all == 3) consume_phase1<3>(p, gr, d, wreg, xreg, lane);
                    else consume_phase1<4>(p, gr, d, wreg, xreg, lane);
                }
            } else {
                // generation g of the operand completes phase g - 1 of its barrier
                ok = mbar_wait(&op_bar, (uint32_t)(d.op_gen - 1) & 1u);
                if (ok) {
                    const int mt = (st_pad8(gr.T) + 15) >> 4;
                    if (mt == 1) consume_phase2<1>(p, gr, d, wreg, oreg, s_slot_token, s_slot_w, lane);
                    else if (mt == 2) consume_phase2<2>(p, gr, d, wreg, oreg, s_slot_token, s_slot_w, lane);
                    else if (mt == 3) consume_phase2<3>(p, gr, d, wreg, oreg, s_slot_token, s_slot_w, lane);
                    else consume_phase2<4>(p, gr, d, wreg, oreg, s_slot_token, s_slot_w, lane);
                }
            }
            if (!ok) {
                if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                break;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[slot]);
        }
    }
}

}  // namespace s2moe
