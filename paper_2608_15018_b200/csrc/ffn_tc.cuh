// tcgen05 expert kernel (kernel plan 3): the selected experts' weights go from HBM to
// shared memory by TMA tensor copies (128-byte swizzle) and from there straight into the
// 5th-generation tensor cores; they never pass through registers.
//
// Both projections are cut into split-K tiles ("units") of equal cost:
//   phase 1 unit: 128 rows of W_gate or W_up of one expert x KT k-tiles of 64
//                 D[row][token] = W[rows, k-range] . h[tokens, k-range]^T       (all B tokens)
//                 -> red.add into pre[slot][gate|up][row]   (only the expert's tokens)
//   phase 2 unit: 128 rows of W_down of one expert x KT k-tiles of 64
//                 D[row][slot] = W[rows, k-range] . a[slots, k-range]^T, a as bf16 hi + lo
//                 -> y[token][row] += p * D                 (red.add, fp32)
// The unit that completes an expert's phase 1 (counter) turns pre into a = silu(g) * u
// (bf16 hi + lo parts) and raises the expert's ready flag, which phase-2 units wait for
// (bounded).  Units are dealt round-robin to one persistent CTA per SM.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (TMEM -> registers -> red.add).  A ring of stages, each one weight
// k-tile (128 x 64 bf16 = 16 KiB) plus the matching token k-tile(s); accumulators are
// double-buffered in TMEM.  tcgen05.mma: M = 128 weight rows, N = tokens padded to 16,
// K = 16 per instruction, fp32 accumulate.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "ffn_stream.cuh"

namespace s2moe {

constexpr int kTcThreads = 192;
constexpr int kTcMaxStages = 12;
constexpr int kTcKT = 4;                       // k-tiles (of 64) per unit: 64 KiB of weights
constexpr int kTcWTile = 128 * 128;            // bytes of one weight k-tile in shared memory
constexpr int kTcMaxSmem = 232448 - 4096;
constexpr unsigned kTcSpinLimit = 1u << 22;
constexpr int kTcReady = 512;                  // ws.sync[kTcReady + a]: activations of active group a are written

struct TcPlan {
    int feasible;
    int n_cta;
    int stages;
    int stage_bytes;   // weight tile + token tiles, multiple of 1024
    int n1;            // tokens padded to 16 (phase-1 N)
    int tmem_cols;     // power of two >= 32
    int tab_bytes;
    int smem_bytes;
};

struct TcArgs {
    Shape sh;
    Workspace ws;
    TcPlan plan;
    float *y;
    float *pre;                       // [slot][2][f_g] fp32 pre-activations (zeroed before the launch)
    __nv_bfloat16 *act_hi, *act_lo;   // [slot][f_g]
    int B;
};

inline TcPlan tc_make_plan(const Shape &sh, int B, int n_sm, int n_slots)
{
    TcPlan p{};
    const int G = sh.E + sh.n_sh;
    p.n_cta = n_sm;
    p.n1 = (B + 15) & ~15;
    // phase-2 stages carry hi and lo tiles of up to n1 slots (a group never has more tokens than B)
    p.stage_bytes = kTcWTile + 2 * p.n1 * 128;
    p.stage_bytes = (p.stage_bytes + 1023) & ~1023;
    p.tab_bytes = ((int)sizeof(StGroup) * (G + 1) + 8 * n_slots + 1023) & ~1023;
    p.stages = (kTcMaxSmem - p.tab_bytes - 1024) / p.stage_bytes;
    if (p.stages > kTcMaxStages) p.stages = kTcMaxStages;
    p.tmem_cols = 32;
    while (p.tmem_cols < 2 * p.n1) p.tmem_cols <<= 1;
    p.smem_bytes = p.tab_bytes + p.stages * p.stage_bytes + 1024;   // + slack to align the ring to 1024
    p.feasible = p.stages >= 4 && B <= kMaxTokens && sh.weight_dtype == DT_BF16 && sh.act_dtype == DT_BF16 &&
                 sh.d % 64 == 0;
    return p;
}

// units of a group: phase 1 = 2 matrices x row blocks x k-pieces, phase 2 = row blocks x k-pieces
__host__ __device__ __forceinline__ int tc_kpieces(int K) { return ((K + 63) / 64 + kTcKT - 1) / kTcKT; }
__host__ __device__ __forceinline__ int tc_units1(int f_g, int d) { return 2 * ((f_g + 127) / 128) * tc_kpieces(d); }
__host__ __device__ __forceinline__ int tc_units2(int f_g, int d) { return ((d + 127) / 128) * tc_kpieces(f_g); }

// ---- PTX helpers (tcgen05, TMA tensor copies) ------------------------------------------

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void tc_ld8(uint32_t taddr, float (&v)[8])
{
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
// K-major, 128-byte swizzle: rows 128 bytes apart, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t tc_smem_desc(const void *p)
{
    const uint64_t addr = (uint64_t)((smem_u32(p) >> 4) & 0x3FFFu);
    return addr | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint32_t tc_idesc(int n)
{
    // D = F32, A = B = BF16, both K-major, N = n, M = 128
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

// Barrier among the four epilogue warps on an mbarrier (count 4), so that the wait is bounded.
__device__ __forceinline__ bool tc_bar(uint64_t *bar, uint32_t &phase, int lane)
{
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    const bool ok = mbar_wait(bar, phase);
    phase ^= 1u;
    return ok;
}

struct TcUnit {
    int phase, a, mat, rb, kt0, kt1;   // group slot, matrix (0 gate, 1 up, 2 down), row block, k-tile range
    int n;                             // MMA N (tokens padded to 16)
};

__device__ __forceinline__ TcUnit tc_decode(const StGroup *groups, int n_active, int total1, int u, int d, int n1)
{
    TcUnit t;
    if (u < total1) {
        t.phase = 1;
        t.a = upper_group1(groups, n_active, u);
        const StGroup &g = groups[t.a];
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
        const StGroup &g = groups[t.a];
        const int local = v - g.p2, kp = tc_kpieces(g.f);
        const int piece = local % kp;
        t.rb = local / kp;
        t.mat = 2;
        t.kt0 = piece * kTcKT;
        t.kt1 = min((g.f + 63) / 64, t.kt0 + kTcKT);
        t.n = (g.T + 15) & ~15;
    }
    return t;
}

// tensor maps: 0 gate, 1 up, 2 down, 3 sh_gate, 4 sh_up, 5 sh_down, 6 hidden, 7/8 act hi/lo routed,
// 9/10 act hi/lo shared
struct TcMaps {
    CUtensorMap m[11];
};

__global__ void __launch_bounds__(kTcThreads, 1) ffn_tc_kernel(const __grid_constant__ TcMaps maps, TcArgs p)
{
    extern __shared__ __align__(1024) uint8_t tc_smem[];
    __shared__ __align__(8) uint64_t full_bar[kTcMaxStages], empty_bar[kTcMaxStages];
    __shared__ __align__(8) uint64_t acc_full[2], acc_empty[2], ep_bar;
    __shared__ uint32_t s_tmem;
    __shared__ int s_flag;

    const Shape &sh = p.sh;
    const Workspace &ws = p.ws;
    const TcPlan &pl = p.plan;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_active = ws.header[0], n_slots = ws.header[1];
    const int G = sh.E + sh.n_sh;

    StGroup *groups = reinterpret_cast<StGroup *>(tc_smem);
    const int tab_rest = pl.tab_bytes - (int)sizeof(StGroup) * (G + 1);
    int *s_slot_token = reinterpret_cast<int *>(tc_smem + sizeof(StGroup) * (G + 1));
    float *s_slot_w = reinterpret_cast<float *>(s_slot_token + tab_rest / 8);
    uint8_t *ring = tc_smem + pl.tab_bytes;
    ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(ring) + 1023) & ~(uintptr_t)1023);

    // group table; stage prefixes follow from the active list alone (routed groups first)
    const int U = ws.header[2];
    const int u1r = tc_units1(sh.f, sh.d), u2r = tc_units2(sh.f, sh.d);
    const int u1s = sh.n_sh ? tc_units1(sh.f_sh, sh.d) : 0, u2s = sh.n_sh ? tc_units2(sh.f_sh, sh.d) : 0;
    for (int a = tid; a < n_active; a += blockDim.x) {
        StGroup gr;
        gr.group = ws.active[a];
        gr.T = ws.counts[gr.group];
        gr.off = ws.offsets[gr.group];
        gr.f = gr.group < sh.E ? sh.f : sh.f_sh;
        gr.mask = ws.tokmask[gr.group];
        const int r = a < U ? a : U, s = a < U ? 0 : a - U;
        gr.p1 = r * u1r + s * u1s;
        gr.p2 = r * u2r + s * u2s;
        gr.nks = 0;
        gr.ksl = 0;
        groups[a] = gr;
    }
    for (int i = tid; i < n_slots; i += blockDim.x) {
        s_slot_token[i] = ws.slot_token[i];
        s_slot_w[i] = ws.slot_w[i];
    }
    const int total1 = U * u1r + sh.n_sh * u1s, total2 = U * u2r + sh.n_sh * u2s;
    const int total = total1 + total2;
    const int S = pl.stages;
    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 4);
        }
        mbar_init(&ep_bar, 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // TMEM: accumulators of two units
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)),
                     "r"((uint32_t)pl.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem;
    const int P = gridDim.x;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            unsigned it = 0;
            bool alive = true;
            for (int u = blockIdx.x; u < total && alive; u += P) {
                const TcUnit t = tc_decode(groups, n_active, total1, u, sh.d, pl.n1);
                const StGroup &g = groups[t.a];
                const bool shared = g.group >= sh.E;
                const int e = shared ? g.group - sh.E : g.group;
                const CUtensorMap *wmap = &maps.m[(shared ? 3 : 0) + t.mat];
                const int rows_per_e = t.mat == 2 ? sh.d : g.f;
                const int row0 = e * rows_per_e + t.rb * 128;
                if (t.phase == 2) {
                    // the expert's activations must have been written
                    bool ok = false;
                    for (unsigned i = 0; i < (kTcSpinLimit >> 2); ++i) {
                        if (ld_acquire(&ws.sync[kTcReady + t.a]) != 0) { ok = true; break; }
                        __nanosleep(40);
                    }
                    if (!ok) { atomicExch(ws.status, ST_DEP_TIMEOUT); alive = false; break; }
                    fence_proxy_async();
                }
                const int n_routed = p.B * sh.k;
                for (int kt = t.kt0; kt < t.kt1; ++kt, ++it) {
                    const int s = it % S;
                    if (!mbar_wait(&empty_bar[s], ((it / S) & 1u) ^ 1u)) {
                        atomicExch(ws.status, ST_MBAR_TIMEOUT);
                        alive = false;
                        break;
                    }
                    uint8_t *stage = ring + (size_t)s * pl.stage_bytes;
                    const uint32_t op_bytes = (uint32_t)t.n * 128u * (t.phase == 1 ? 1u : 2u);
                    mbar_expect_tx(&full_bar[s], kTcWTile + op_bytes);
                    tma_load_2d(stage, wmap, kt * 64, row0, &full_bar[s]);
                    uint8_t *op = stage + kTcWTile;
                    if (t.phase == 1) {
                        for (int r = 0; r < t.n; r += 16) tma_load_2d(op + r * 128, &maps.m[6], kt * 64, r, &full_bar[s]);
                    } else {
                        const int srow = shared ? g.off - n_routed : g.off;   // row in the routed / shared act array
                        const CUtensorMap *hi = &maps.m[shared ? 9 : 7], *lo = &maps.m[shared ? 10 : 8];
                        for (int r = 0; r < t.n; r += 16) {
                            tma_load_2d(op + r * 128, hi, kt * 64, srow + r, &full_bar[s]);
                            tma_load_2d(op + (t.n + r) * 128, lo, kt * 64, srow + r, &full_bar[s]);
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            unsigned it = 0, ui = 0;
            bool alive = true;
            for (int u = blockIdx.x; u < total && alive; u += P, ++ui) {
                const TcUnit t = tc_decode(groups, n_active, total1, u, sh.d, pl.n1);
                const int buf = ui & 1;
                if (!mbar_wait(&acc_empty[buf], ((ui >> 1) & 1u) ^ 1u)) {
                    atomicExch(ws.status, ST_MBAR_TIMEOUT);
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * pl.n1);
                const uint32_t idesc = tc_idesc(t.n);
                uint32_t acc = 0;
                for (int kt = t.kt0; kt < t.kt1; ++kt, ++it) {
                    const int s = it % S;
                    if (!mbar_wait(&full_bar[s], (it / S) & 1u)) {
                        atomicExch(ws.status, ST_MBAR_TIMEOUT);
                        alive = false;
                        break;
                    }
                    tc_fence_after();
                    const uint8_t *stage = ring + (size_t)s * pl.stage_bytes;
                    const uint64_t ad = tc_smem_desc(stage);
                    const uint64_t bd = tc_smem_desc(stage + kTcWTile);
                    const uint64_t ld = tc_smem_desc(stage + kTcWTile + t.n * 128);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {      // 4 x K=16 inside the 64-wide tile: +32 bytes each
                        tc_mma_bf16(d_tmem, ad + 2 * k, bd + 2 * k, idesc, acc);
                        acc = 1;
                        if (t.phase == 2) tc_mma_bf16(d_tmem, ad + 2 * k, ld + 2 * k, idesc, 1);
                    }
                    tc_commit(&empty_bar[s]);          // frees the stage when these MMAs have read it
                }
                if (alive) tc_commit(&acc_full[buf]);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;                        // TMEM lane quarter this warp may read
        unsigned ui = 0;
        uint32_t ep_phase = 0;
        const int n_routed = p.B * sh.k;
        bool alive = true;
        for (int u = blockIdx.x; u < total && alive; u += P, ++ui) {
            const TcUnit t = tc_decode(groups, n_active, total1, u, sh.d, pl.n1);
            const StGroup &g = groups[t.a];
            const int buf = ui & 1;
            if (!mbar_wait(&acc_full[buf], (ui >> 1) & 1u)) {
                if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                break;
            }
            tc_fence_after();
            const int row = t.rb * 128 + q * 32 + lane;           // row of the matrix inside the expert
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * pl.n1);
            if (t.phase == 1) {
                const bool row_ok = row < g.f;
                for (int c = 0; c < t.n; c += 8) {
                    float v[8];
                    tc_ld8(taddr + c, v);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int b = c + i;
                        if (b < p.B && ((g.mask >> b) & 1ull) && row_ok) {
                            const int slot = g.off + __popcll(g.mask & ((1ull << b) - 1ull));
                            atomicAdd(&p.pre[2 * act_offset(slot, n_routed, sh.f, sh.f_sh) + (size_t)t.mat * g.f + row], v[i]);
                        }
                    }
                }
            } else {
                const bool row_ok = row < sh.d;
                for (int c = 0; c < t.n; c += 8) {
                    float v[8];
                    tc_ld8(taddr + c, v);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int ti = c + i;
                        if (ti < g.T && row_ok) {
                            const int slot = g.off + ti;
                            atomicAdd(&p.y[(size_t)s_slot_token[slot] * sh.d + row], s_slot_w[slot] * v[i]);
                        }
                    }
                }
            }
            // the accumulator may be overwritten
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            if (t.phase == 1) {
                // count the unit; whoever completes the expert's phase 1 writes its activations
                __threadfence();
                if (!tc_bar(&ep_bar, ep_phase, lane)) { alive = false; break; }
                if (warp == 2 && lane == 0) {
                    const int done = atomicAdd(&ws.sync[t.a], 1) + 1;
                    s_flag = done == tc_units1(g.f, sh.d);
                }
                if (!tc_bar(&ep_bar, ep_phase, lane)) { alive = false; break; }
                if (s_flag) {
                    __threadfence();
                    const int et = tid - 64;                      // 0..127
                    for (int i = et; i < g.T * g.f; i += 128) {
                        const int ti = i / g.f, j = i - ti * g.f;
                        const size_t o = act_offset(g.off + ti, n_routed, sh.f, sh.f_sh);
                        const float gv = __ldcg(&p.pre[2 * o + j]), uv = __ldcg(&p.pre[2 * o + g.f + j]);
                        const float a = silu_mul(gv, uv);
                        const __nv_bfloat16 hi = __float2bfloat16_rn(a);
                        p.act_hi[o + j] = hi;
                        p.act_lo[o + j] = __float2bfloat16_rn(a - __bfloat162float(hi));
                    }
                    __threadfence();
                    fence_proxy_async();
                    if (!tc_bar(&ep_bar, ep_phase, lane)) { alive = false; break; }
                    if (warp == 2 && lane == 0) atomicExch(&ws.sync[kTcReady + t.a], 1);
                }
            }
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

}  // namespace s2moe
