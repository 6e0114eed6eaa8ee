// tcgen05 expert kernel (kernel plan 3): the selected experts' weights go from HBM to
// shared memory by TMA tensor copies (128-byte swizzle) and from there straight into the
// 5th-generation tensor cores; they never pass through registers.
//
// Both projections are cut into split-K tiles ("units") of equal cost:
//   phase 1 unit: 128 rows of W_gate or W_up of one expert x KT k-tiles of 64
//                 D[row][token] = W[rows, k-range] . h[tokens, k-range]^T       (all B tokens)
//                 -> red.add into pre[gate|up][slot][row]   (only the expert's tokens)
//   phase 2 unit: 128 rows of W_down of one expert x KT k-tiles of 64
//                 D[row][slot] = W[rows, k-range] . a[slots, k-range]^T, a as bf16 hi + lo
//                 -> y[token][row] += p * D                 (red.add, fp32)
// The experts are split into two waves.  When a CTA has finished its phase-1 units of a wave
// its epilogue hands the wave over to the CTA's converter warps, which arrive on the wave's
// grid-wide counter, wait (bounded) until all CTAs have arrived, turn their slice of the wave's
// pre into a = silu(g) * u (bf16 hi + lo parts) and arrive on the wave's second counter, which
// the phase-2 token tiles of that wave wait for.  So the hand-over between the projections
// of one wave hides behind the other wave's work.  One persistent CTA per SM; of each of the
// four segments (phase 1 / 2 of wave 0 / 1) a CTA takes one contiguous run of units, so that
// consecutive k-pieces of a row block accumulate in TMEM and are reduced to memory once.
//
// Warp roles (352 threads): warp 0 = TMA producer; warps 1 and 6 = MMA issuers (warp 1 owns the
// TMEM allocation); warps 2..5 = epilogue (TMEM -> registers -> red.add); warps 7..9 = converters;
// warp 10 = watcher (polls the waves' second counters and publishes them in shared memory, so
// that the producer never waits on global memory).  A ring of stages, each one weight k-tile
// (128 x 64 bf16 = 16 KiB) plus the matching token k-tiles (phase 1: hidden states; phase 2: per
// 8 slots their hi rows and, right behind, their lo rows); accumulators are double-buffered in
// TMEM.  tcgen05.mma: M = 128 weight rows, N = 16 per 16 tokens (phase 1) or per 8 hi + lo slots
// (phase 2), K = 16 per instruction, fp32 accumulate.
//
// Block-int4 weights (template parameter): the ring holds packed tiles and scales, up to a whole
// unit per stage, and eight more warps dequantise every stage into a second ring of bf16 tiles that
// the MMA issuers read (four of them where the accumulators fit); the token tiles of a stage are
// fetched into a slot of that second ring, so a packed stage is free as soon as it has been read.
// See the producer's int4 branch and the dequantising branch below.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "ffn_stream.cuh"

namespace s2moe {

constexpr int kTcThreads = 352;                // warps: producer, MMA issuer 0, 4 epilogue, MMA issuer 1, 4 converters
// block-int4 weights: warps that dequantise (8 or 16: 4 or 2 chunks of a row per thread).  The path is
// bound by the instructions it issues, and 16 warps spend more of them on waiting and signalling
// than they gain in latency hiding (measured: 156 us against 145 us per layer of the Mixtral shape).
constexpr int kTcQ4DeqWarps = 8;
constexpr int kTcQ4Threads = kTcThreads + 32 * kTcQ4DeqWarps + 64;   // ... and two more MMA issuers behind them
constexpr int kTcQ4Packed = 128 * 32;          // bytes of one packed weight k-tile (128 rows x 64 nibbles)
constexpr int kTcQ4Scales = 128 * 16;          // 8 binary16 scales per row: the 256 columns of the tile's unit
constexpr int kTcMaxAStages = 6;               // stages of dequantised bf16 weight tiles
constexpr int kTcQ4KG = 4;                     // int4: k-tiles per stage (a whole unit)
static_assert(kTcQ4KG == 4, "the int4 path takes a stage to be a whole unit of four k-tiles");
constexpr int kTcQ4ACol = 256;                 // int4: TMEM columns 256.. hold the dequantised tiles (32 per k-tile), 0..255 the accumulators
#ifndef S2MOE_MAX_STAGES
#define S2MOE_MAX_STAGES 10
#endif
constexpr int kTcMaxStages = S2MOE_MAX_STAGES;  // barrier arrays; the int4 ring
constexpr int kTcRingDepth = 8;                // bf16 weights: stages of the ring at most (see tc_make_plan)
constexpr int kTcMinStagesResident = 6;        // bf16 weights: the hidden-state tiles stay in shared memory if this many stages fit beside them
constexpr int kTcKT = 4;                       // k-tiles (of 64) per unit: 64 KiB of weights
constexpr int kTcWTile = 128 * 128;            // bytes of one weight k-tile in shared memory
constexpr int kTcMaxSmem = 232448 - 9216;      // dynamic shared memory; the rest is static (unit table, barriers)
constexpr unsigned kTcSpinLimit = 1u << 22;
constexpr int kTcMaxWaves = 3;                 // waves the experts are cut into at most (see the kernel)
constexpr int kTcMaxAcc = 8;                   // accumulator buffers in tensor memory (2 without the early start)
constexpr int kTcMaxUnits = 192;               // units of one CTA decoded once into shared memory
// Share of the experts in wave 0 (by units of the first projection).  The second projection of
// wave 0 is what hides the hand-over of wave 1, the first projection of wave 1 what hides that of
// wave 0.  Measured with the kernel as it stands (early start, two k-tiles per stage), us per layer
// at 6 / 7 / 8 / 9 / 10 / 11 sixteenths: OLMoE shape at 8 tokens 49.98 / 49.87 / 49.67 / 49.93 /
// 49.94 / 50.41, DeepSeek-V2-Lite shape at 16 tokens 59.65 / 59.19 / 59.07 / 59.13 / 60.74 / 62.13,
// Qwen1.5-MoE shape at 16 tokens 54.45 / 54.60 / 55.16 / 56.01 / 56.96 / 57.17; one wave: 52.8, 64.6,
// 57.2; three waves (5 and 11, 4 and 10 sixteenths): 52.2 to 52.9 at the OLMoE shape (every
// hand-over costs two grid-wide rounds and cuts accumulation runs), 58.6 to 58.8 at DeepSeek-V2-Lite.
#ifndef S2MOE_SPLIT_NUM
#define S2MOE_SPLIT_NUM 7
#define S2MOE_SPLIT_DEN 16
#endif
constexpr int kTcSplitNum = S2MOE_SPLIT_NUM, kTcSplitDen = S2MOE_SPLIT_DEN;
constexpr int kTcReady = 512;                  // ws.sync[kTcReady - 8 + w], [kTcReady - 4 + w]: the two counters of wave w

// one active group in shared memory: 32 bytes, so that an entry is two aligned 16-byte reads
// (wider entries were measured: 48 bytes cost 0.7 us per layer)
struct TcGroup {
    unsigned long long mask;   // tokens of the batch bucketed to this group
    int group, T, off, f;      // group id (offloaded experts: device slot), tokens, first slot, inner dim
    int p1, p2;                // first phase-1 / phase-2 unit of the group
};
static_assert(sizeof(TcGroup) == 32, "layout");

struct TcPlan {
    int feasible;
    int n_cta;
    int stages;
    int stage_bytes;   // weight tile + token tiles, multiple of 1024
    int n1;            // tokens padded to 16 (phase-1 N)
    int tmem_cols;     // power of two >= 32
    int n_iss;         // MMA issuer warps (2, or 4 on the int4 path when the accumulators fit)
    int tab_bytes;
    int x_bytes;       // > 0: the hidden states stay resident in shared memory (all k-tiles)
    int smem_bytes;
    int q4;            // block-int4 weights: packed tiles in the ring, dequantised into a second ring
    int a_stages;      // stages of that second ring
    int tok_off;       // offset of the token tiles inside a stage
    int kg;            // k-tiles per stage (1 for bf16 weights; 1, 2 or 4 for int4)
    int tokb;          // bytes of the token tiles of one k-tile
    int rows1;         // rows of one hidden-state copy (bf16, one k-tile per stage)
    int n_acc;         // accumulator buffers (a power of two; more than 2 only with the early start)
    int early;         // the early start is possible for this shape (bf16 weights, units fit the table)
    int split[2];      // where wave 1 and wave 2 begin, in 16ths of the first projection's units (16: no such wave)
};

struct TcArgs {
    Shape sh;
    Workspace ws;
    TcPlan plan;
    float *y;
    float *pre;                       // [gate|up][slot][f_g] fp32 pre-activations (zeroed by the routing kernel)
    __nv_bfloat16 *act_hi, *act_lo;   // [slot][f_g]
    int B;
    int early;                        // 1: early start (see the kernel)
};

// units of a group: phase 1 = 2 matrices x row blocks x k-pieces, phase 2 = row blocks x k-pieces
__host__ __device__ __forceinline__ int tc_kpieces(int K) { return ((K + 63) / 64 + kTcKT - 1) / kTcKT; }
__host__ __device__ __forceinline__ int tc_units1(int f_g, int d) { return 2 * ((f_g + 127) / 128) * tc_kpieces(d); }
__host__ __device__ __forceinline__ int tc_units2(int f_g, int d) { return ((d + 127) / 128) * tc_kpieces(f_g); }

inline TcPlan tc_make_plan(const Shape &sh, int B, int n_sm, int n_slots, int bf16_kg = 2, bool early = false)
{
    TcPlan p{};
    const int G = sh.E + sh.n_sh;
    p.n_cta = n_sm;
    p.n1 = (B + 15) & ~15;
    // token area of a stage: phase 1 = n1 rows of 128 bytes; phase 2 = per 8 slots their hi rows
    // (1 KiB) and right behind them their lo rows (a group never has more tokens than B)
    p.stage_bytes = kTcWTile + 2048 * ((B + 7) / 8);
    p.stage_bytes = (p.stage_bytes + 1023) & ~1023;
    p.tab_bytes = ((int)sizeof(TcGroup) * (G + 1 + sh.n_sh) + 8 * n_slots + 1023) & ~1023;
    // Shared memory between the ring and the hidden-state tiles (bf16 weights).  Measured with the
    // early start in place (OLMoE, Qwen1.5-MoE and DeepSeek-V2-Lite shapes, 4 to 16 tokens): a ring of
    // 6 to 8 stages with the hidden-state tiles resident (the first projection's stages then take one
    // copy instead of two) beats 10 stages without them by 1.3 to 1.8 us per layer, 5 stages lose
    // 0.1 to 0.3 us again, and 8 stages without resident tiles are no slower than 10.  So the tiles
    // stay resident wherever 6 stages fit beside them, and the ring is never deeper than 8.
    p.x_bytes = ((sh.d + 63) / 64) * p.n1 * 128;
    if ((kTcMaxSmem - p.tab_bytes - 1024 - p.x_bytes) / p.stage_bytes < kTcMinStagesResident) p.x_bytes = 0;
    p.stages = (kTcMaxSmem - p.tab_bytes - 1024 - p.x_bytes) / p.stage_bytes;
    if (p.stages > kTcRingDepth) p.stages = kTcRingDepth;
    p.n_iss = 2;
    p.tmem_cols = 32;
    while (p.tmem_cols < 8 * p.n1) p.tmem_cols <<= 1;   // 2 buffers x 2 issuers x up to 2 * n1 columns
    p.smem_bytes = p.tab_bytes + p.x_bytes + p.stages * p.stage_bytes + 1024;   // + slack to align to 1024
    p.tok_off = kTcWTile;
    p.kg = 1;
    p.tokb = 2048 * ((B + 7) / 8);
    p.rows1 = p.n1;    // the hidden-state k-tile of a stage in ONE copy (the producer is a single thread)
    // bf16 weights: TWO k-tiles per ring stage where every contraction length is a multiple of 64
    // (one weight copy of 32 KiB and one token copy per stage, one barrier round trip and five
    // instead of six tensor-core instructions per issuer and 32 KiB).  The producer and the MMA
    // issuers are single threads whose instructions cost tens of cycles each, and at 6 TB/s a
    // 16 KiB k-tile has to leave an SM every 400 ns: with one k-tile per stage those loops are at
    // their limit.  Measured (us per layer, one / two k-tiles per stage, resident hidden-state tiles
    // in both where they fit): OLMoE shape 8 tokens 48.6 / 48.3, 16 tokens 55.7 / 53.6, 24 tokens
    // 63.6 / 60.6; Qwen1.5-MoE shape 16 tokens 58.2 / 54.8; DeepSeek-V2-Lite shape 16 tokens 62.3 /
    // 58.2, 64 tokens 121 / 109 (before the early start); a single token: 38.1 / 38.6, so the caller
    // asks for it from two tokens on.  Three such stages beside the resident tiles beat five
    // without them.
    if (bf16_kg == 2 && sh.weight_dtype == DT_BF16 && sh.d % 64 == 0 && sh.f % 64 == 0 && (sh.n_sh == 0 || sh.f_sh % 64 == 0)) {
        p.kg = 2;
        p.stage_bytes = (2 * kTcWTile + 2 * p.tokb + 1023) & ~1023;
        p.tok_off = 2 * kTcWTile;
        // (resident hidden-state tiles as above, if 3 of these stages fit beside them and no stage
        // reaches past the last k-tile)
        p.x_bytes = ((sh.d / 64) % 2 == 0) ? (sh.d / 64) * p.n1 * 128 : 0;
        if ((kTcMaxSmem - p.tab_bytes - 1024 - p.x_bytes) / p.stage_bytes < 3) p.x_bytes = 0;
        p.stages = (kTcMaxSmem - p.tab_bytes - 1024 - p.x_bytes) / p.stage_bytes;
        if (p.stages > kTcRingDepth) p.stages = kTcRingDepth;
        p.smem_bytes = p.tab_bytes + p.x_bytes + p.stages * p.stage_bytes + 1024;
        if (p.stages < 3) {          // (large batches: back to one k-tile per stage)
            p.kg = 1;
            p.x_bytes = 0;
            p.stage_bytes = (kTcWTile + p.tokb + 1023) & ~1023;
            p.tok_off = kTcWTile;
            p.stages = (kTcMaxSmem - p.tab_bytes - 1024) / p.stage_bytes;
            if (p.stages > kTcMaxStages) p.stages = kTcMaxStages;
            p.smem_bytes = p.tab_bytes + p.stages * p.stage_bytes + 1024;
        }
    }
    p.n_acc = 2;
    p.early = 0;
    p.split[0] = kTcSplitNum * 16 / kTcSplitDen;
    p.split[1] = 16;
    if (early && sh.weight_dtype == DT_BF16 && n_sm > 1) {
        // Early start (see the kernel): one CTA less than SMs, because the SM that runs the gating is
        // taken until the routing kernel ends and its CTA would start last with a full share; as many
        // accumulators as tensor memory holds (the reductions of an early expert wait for the
        // tables); and only where a CTA's units are sure to fit the table in shared memory.
        const int P = n_sm - 1;
        const long long worst = (long long)sh.E * (tc_units1(sh.f, sh.d) + tc_units2(sh.f, sh.d)) +
                                (long long)sh.n_sh * (tc_units1(sh.f_sh, sh.d) + tc_units2(sh.f_sh, sh.d));
        if (worst / P + 12 <= kTcMaxUnits) {
            p.early = 1;
            p.n_cta = P;
            int nb = 8;
            while (nb > 2 && nb * 4 * p.n1 > 512) nb >>= 1;
            p.n_acc = nb;
            p.tmem_cols = 32;
            while (p.tmem_cols < nb * 4 * p.n1) p.tmem_cols <<= 1;
        }
    }
    p.feasible = p.stages >= (p.kg == 2 ? 3 : 4) && B <= kMaxTokens && sh.weight_dtype == DT_BF16 && sh.act_dtype == DT_BF16 &&
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


// ---- PTX helpers (tcgen05, TMA tensor copies) ------------------------------------------

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
// Weight tiles are read once: mark their L2 lines evict-first, so that the stream does not push
// out what is reused across layers (kernel code, bucketing arrays, activations).
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_load_2d_stream(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar,
                                                   uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_stream(void *dst, const CUtensorMap *map, int x, int y, int z, uint64_t *bar,
                                                   uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4, %5}], [%2], %6;"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int x, int y, int z, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, int x, int y, int z, int w, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}
// (x & mask) | bits in one logic instruction
__device__ __forceinline__ void tc_nibble_pair(uint32_t &out, uint32_t x, uint32_t mask, uint32_t bits)
{
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(out) : "r"(x), "r"(mask), "r"(bits));
}
// non-blocking test of a phase (a thread that serves two rings polls both)
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
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
// The same with the two descriptors given as their 32-bit halves: the shared-memory address sits in
// the low 14 bits of the low word (in units of 16 bytes), so stepping from tile to tile is one
// 32-bit add.  The issuing thread shares its scheduler with busy warps, and every instruction it
// needs per MMA delays the MMA.
__device__ __forceinline__ void tc_mma_bf16_parts(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                  uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        ".reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, {%7, %7, %7, %7}, p;\n\t"
        "}\n" ::"r"(d_tmem),
        "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// A operand in tensor memory (row i of the 128 x 16 tile in lane i, two bf16 per 32-bit column)
__device__ __forceinline__ void tc_mma_bf16_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                                   uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        ".reg .b64 db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, {%6, %6, %6, %6}, p;\n\t"
        "}\n" ::"r"(d_tmem),
        "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// 16 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
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
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// K-major, 128-byte swizzle: rows 128 bytes apart, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t tc_smem_desc(const void *p)
{
    const uint64_t addr = (uint64_t)((smem_u32(p) >> 4) & 0x3FFFu);
    return addr | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// the same with 8-row groups `sbo` bytes apart
__device__ __forceinline__ uint64_t tc_smem_desc_sbo(const void *p, uint32_t sbo)
{
    const uint64_t addr = (uint64_t)((smem_u32(p) >> 4) & 0x3FFFu);
    return addr | (1ull << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint32_t tc_idesc(int n)
{
    // D = F32, A = B = BF16, both K-major, N = n, M = 128
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ uint32_t tc_idesc_f16(int n)
{
    // the same with A = B = binary16 (int4 path: the dequantised weights and, because the two
    // operands of an instruction must have one format, the token tiles as well)
    return (1u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
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

// counter += 1 with release semantics at GPU scope (one instruction instead of fence + atomic)
__device__ __forceinline__ void tc_red_release(int32_t *counter)
{
    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(counter) : "memory");
}

// next slot of the ring; the parity flips on wrap-around
__device__ __forceinline__ void tc_ring_next(int &s, uint32_t &parity, int S)
{
    if (++s == S) { s = 0; parity ^= 1u; }
}

struct TcUnit {                        // plain ints: the single-thread roles read these on their critical path
    int phase, a, mat, rb, kt0, kt1;   // group slot, matrix (0 gate, 1 up, 2 down), row block, k-tile range
    int n;                             // MMA N: phase 1 tokens padded to 16; phase 2 16 per 8 slots (hi | lo)
    int seg;                           // 0 / 1: phase 1 of wave 0 / 1, 2 / 3: phase 2 of wave 0 / 1
    int first, last;                   // first / last unit of an accumulation run (see the kernel)
};

__device__ __forceinline__ TcUnit tc_decode(const TcGroup *groups, int n_active, int total1, int u, int d, int n1)
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
__device__ __forceinline__ uint32_t tc_unit_meta(const TcUnit &t)
{
    return (uint32_t)t.first | ((uint32_t)t.last << 1) | ((t.phase == 2 ? 1u : 0u) << 2) | ((uint32_t)t.n << 8);
}

// tensor maps: 0 gate, 1 up, 2 down, 3 sh_gate, 4 sh_up, 5 sh_down, 6 hidden, 7 activations of the
// routed slots, 8 of the shared slots: 3-D {k, slot, hi|lo}, so that one copy of box {64, 16, 2}
// lands the hi tile and, right behind it, the lo tile of 16 slots
// block-int4 weights: 0..5 are the packed matrices (bytes) with a box of one k-tile, 9..14 their
// scales (binary16), 15..20 and 21..26 the packed matrices again with boxes of two and four k-tiles;
// 6 is the (column-permuted) hidden states as {k in tile, row, k-tile} with a box of all rows x kg
// k-tiles, 7 and 8 the activations as {k in tile, slot, k-tile, hi|lo} with a box {64, 8, kg, 2}:
// one copy per stage (per 8 slots) instead of one per k-tile
struct TcMaps {
    CUtensorMap m[27];
};

template <bool Q4>
__global__ void __launch_bounds__(Q4 ? kTcQ4Threads : kTcThreads, 1)
ffn_tc_kernel(const __grid_constant__ TcMaps maps, TcArgs p)
{
    extern __shared__ __align__(1024) uint8_t tc_smem[];
    __shared__ __align__(8) uint64_t full_bar[kTcMaxStages], empty_bar[kTcMaxStages];
    __shared__ __align__(8) uint64_t acc_full[kTcMaxAcc], acc_empty[kTcMaxAcc], ep_bar, x_bar, cv_bar, conv_go[kTcMaxWaves], tab_bar;
    __shared__ __align__(8) uint64_t a_full[kTcMaxAStages], a_empty[kTcMaxAStages];   // int4: dequantised tiles
    __shared__ uint32_t s_tmem;
    __shared__ int s_flag;
    __shared__ TcUnit s_units[kTcMaxUnits];
    __shared__ uint32_t s_umeta[kTcMaxUnits];      // what an MMA issuer needs of a unit, in one word (tc_unit_meta)
    __shared__ int s_split[2];                     // first active group of wave 1 and of wave 2 (n_active: no such wave)
    __shared__ unsigned s_early32[8];              // early start: the routing kernel's list of early experts, 32 per word
    __shared__ int s_tab[2];                       // early start: units of the routed work of this CTA, active groups
    __shared__ volatile int s_ready[kTcMaxWaves];  // wave w's activations are written (set by the watcher warp)

    const Shape &sh = p.sh;
    const Workspace &ws = p.ws;
    const TcPlan &pl = p.plan;
    const int NI = Q4 ? p.plan.n_iss : 2;          // MMA issuers: a compile-time 2 on the bf16 path
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // Set-up that needs nothing of the routing kernel comes first: this grid is launched
    // programmatically, so its CTAs may become resident while the routing kernel still runs
    if (warp == 2) {
        // barrier set-up, spread over a warp so that it runs beside the table loads of the others
        if (lane < pl.stages) {
            mbar_init(&full_bar[lane], 1);
            mbar_init(&empty_bar[lane], Q4 ? kTcQ4DeqWarps : NI);   // one commit from each MMA issuer; int4: the dequantising warps
        }
        if (lane < kTcMaxAcc) {
            mbar_init(&acc_full[lane], NI);
            mbar_init(&acc_empty[lane], 4);
        }
        if (lane < kTcMaxWaves) mbar_init(&conv_go[lane], 4);
        if (Q4 && lane < pl.a_stages) {
            mbar_init(&a_full[lane], kTcQ4DeqWarps + 1);   // the dequantising warps and the producer's arrival with the token bytes
            mbar_init(&a_empty[lane], NI);
        }
        if (lane == 0) {
            mbar_init(&ep_bar, 4);
            mbar_init(&x_bar, 1);
            mbar_init(&cv_bar, 3);
            mbar_init(&tab_bar, 1);
            s_ready[0] = 0;
            s_ready[1] = 0;
            s_ready[2] = 0;
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
    // Early start (bf16 weights, see tc_make_plan): this grid does not wait for the routing kernel
    // as a whole.  The routing kernel publishes, before its gating, the experts that are certain
    // to be selected; their first projection and that of the shared experts (the "pre-lot") is
    // streamed while the gating runs.  Warps 7..10, idle until the first hand-over, wait for the
    // routing kernel to end, build the tables of everything else and open tab_bar; the other
    // roles pass that barrier when they have worked off their share of the pre-lot.
    const bool EARLY = !Q4 && p.early != 0;
    const int n_slots = p.B * sh.k + sh.n_sh * p.B;          // every token fills k routed slots
    const int G = sh.E + sh.n_sh;
    const int GP = G + 1;                                    // early start: provisional groups of the shared experts

    TcGroup *groups = reinterpret_cast<TcGroup *>(tc_smem);
    const int n_tab_groups = G + 1 + sh.n_sh;
    const int tab_rest = pl.tab_bytes - (int)sizeof(TcGroup) * n_tab_groups;
    int *s_slot_token = reinterpret_cast<int *>(tc_smem + sizeof(TcGroup) * n_tab_groups);
    float *s_slot_w = reinterpret_cast<float *>(s_slot_token + tab_rest / 8);
    uint8_t *xres = tc_smem + pl.tab_bytes;
    xres = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(xres) + 1023) & ~(uintptr_t)1023);
    uint8_t *ring = xres + pl.x_bytes;
    uint8_t *tokring = ring + (size_t)pl.stages * pl.stage_bytes;    // int4 only: token tiles, one slot per slot of dequantised tiles

    const int u1r = tc_units1(sh.f, sh.d), u2r = tc_units2(sh.f, sh.d);
    const int u1s = sh.n_sh ? tc_units1(sh.f_sh, sh.d) : 0, u2s = sh.n_sh ? tc_units2(sh.f_sh, sh.d) : 0;
    const int S = pl.stages;
    const int P = gridDim.x;
    // Where every unit of a projection has all its four k-tiles (contraction length a multiple of
    // 256) the segments are dealt in half units, so that the CTAs of a segment differ by two
    // k-tiles (0.75 us) instead of four: a share may then begin with the second half of a unit
    // and end with the first half of one (trim bits 1 and 2).  Measured at the OLMoE shape: 0.7 %
    // of a layer; dealing single k-tiles cuts more accumulation runs in two and gives it back.
    // The int4 path needs whole units.
    const bool halves1 = !Q4 && sh.d % 256 == 0;
    const bool halves2 = !Q4 && sh.f % 256 == 0 && (sh.n_sh == 0 || sh.f_sh % 256 == 0);
    // Every CTA takes one contiguous run of units of each segment (sizes differ by at most one;
    // the CTAs that get the extra unit rotate from segment to segment, so the totals differ by at
    // most one as well).
    int rot = 0;
    auto share = [&](int begin, int n, bool halves, int &start, int &cnt, int &trim) {
        const int m = halves ? 2 : 1, n2 = n * m;
        const int q = n2 / P, r = n2 - q * P;
        int c = (int)blockIdx.x - rot;               // (blockIdx.x - rot) mod P without a division:
        if (c < 0) c += P;                           // the calls would otherwise chain as many of them
        const int cnt2 = q + (c < r ? 1 : 0), start2 = c * q + min(c, r);
        const int u0 = halves ? start2 >> 1 : start2, u1 = halves ? (start2 + cnt2 - 1) >> 1 : start2 + cnt2 - 1;
        cnt = cnt2 > 0 ? u1 - u0 + 1 : 0;
        start = begin + u0;
        trim = (halves && cnt2 > 0) ? ((start2 & 1) | (((start2 + cnt2) & 1) << 1)) : 0;
        rot += r;
        if (rot >= P) rot -= P;
    };

    // ---- the pre-lot (early start only)
    int n_early = 0, n_pre = 0, pre_start = 0, pre_trim = 0;
    if (EARLY) {
        if (warp == 0) {
            // bounded wait for the routing kernel's list: one tagged 64-bit word per 32 experts, each
            // polled by a lane of its own (a release store behind everything that kernel clears; all
            // its blocks are resident or done when this grid is scheduled)
            const int nwords = (sh.E + 31) >> 5;
            unsigned long long v = 0ull;
            bool ok = false;
            for (unsigned i = 0; i < (1u << 21); ++i) {
                if (lane < nwords)
                    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(reinterpret_cast<const unsigned long long *>(ws.early) + lane) : "memory");
                if (__all_sync(0xffffffffu, lane >= nwords || (v >> 32) == 1ull)) { ok = true; break; }
                __nanosleep(20);
            }
            if (lane < 8) s_early32[lane] = (ok && lane < nwords) ? (unsigned)v : 0u;
            if (lane == 0) {
                if (!ok) atomicExch(ws.status, ST_DEP_TIMEOUT);
                s_flag = ok;
            }
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        unsigned ew[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) { ew[q] = s_early32[q]; n_early += __popc(ew[q]); }
        n_early = min(n_early, min(p.B, sh.E));
        const unsigned long long all = p.B >= 64 ? ~0ull : ((1ull << p.B) - 1ull);
        // provisional groups: a shared expert's is complete (every token, slots known); an early
        // routed expert's sits where its final entry will be (the early experts lead the active
        // list in this order) and has only what the producer and the MMA issuers need
        for (int j = tid; j < n_early + sh.n_sh; j += blockDim.x) {
            TcGroup gr;
            if (j < n_early) {
                // the j-th expert of the list: its word first, then its bit by clearing the rem bits below it
                int rem = j, wq = 0;
                unsigned wbits = ew[0];
#pragma unroll
                for (int q = 0; q < 7; ++q) {
                    const int c = __popc(ew[q]);
                    if (wq == q && rem >= c) { rem -= c; wq = q + 1; wbits = ew[q + 1]; }
                }
                for (int t = 0; t < rem; ++t) wbits &= wbits - 1u;
                const int id = 32 * wq + __ffs(wbits) - 1;
                gr.mask = 0ull; gr.group = id; gr.T = 0; gr.off = 0; gr.f = sh.f;
                gr.p1 = sh.n_sh * u1s + j * u1r; gr.p2 = 0;
                groups[j] = gr;
            } else {
                const int sx = j - n_early;
                gr.mask = all; gr.group = sh.E + sx; gr.T = p.B; gr.off = p.B * sh.k + sx * p.B; gr.f = sh.f_sh;
                gr.p1 = sx * u1s; gr.p2 = 0;
                groups[GP + sx] = gr;
            }
        }
        share(0, sh.n_sh * u1s + n_early * u1r, halves1, pre_start, n_pre, pre_trim);
        if (n_pre > kTcMaxUnits) {                    // (the host leaves the early start off where this could happen)
            if (tid == 0) atomicExch(ws.status, ST_BAD_PLAN);
            n_pre = kTcMaxUnits;
        }
    }
    // unit i of this CTA's share of the pre-lot: shared experts first (their reductions need no table)
    auto pre_unit_make = [&](int i) -> TcUnit {
        const int u = pre_start + i, kt_all = (sh.d + 63) / 64;
        TcUnit t;
        int local, f_g;
        if (u < sh.n_sh * u1s) { const int sx = u / u1s; t.a = GP + sx; local = u - sx * u1s; f_g = sh.f_sh; }
        else { const int v = u - sh.n_sh * u1s, j = v / u1r; t.a = j; local = v - j * u1r; f_g = sh.f; }
        const int kp = tc_kpieces(sh.d), rbs = (f_g + 127) / 128;
        const int piece = local % kp, rest = local / kp;
        t.phase = 1;
        t.rb = rest % rbs;
        t.mat = rest / rbs;
        t.kt0 = piece * kTcKT;
        t.kt1 = min(kt_all, t.kt0 + kTcKT);
        t.n = pl.n1;
        if (i == 0 && (pre_trim & 1)) t.kt0 += kTcKT / 2;
        if (i == n_pre - 1 && (pre_trim & 2)) t.kt1 -= kTcKT / 2;
        t.seg = 0;
        t.first = (i == 0 || t.kt0 == 0) ? 1 : 0;
        t.last = (i == n_pre - 1 || t.kt1 == kt_all) ? 1 : 0;
        return t;
    };
    if (EARLY) {
        for (int i = tid; i < n_pre; i += blockDim.x) {
            const TcUnit t = pre_unit_make(i);
            s_units[i] = t;
            s_umeta[i] = tc_unit_meta(t);
        }
        __syncthreads();
    }

    // ---- the tables of the routed work: by every thread of the CTA (tt, tn = thread, threads; hardware
    // barrier 0) or, with the early start, by warps 7..10 alone (barrier 1)
    int n_active = 0, U = 0, total1 = 0, total2 = 0, a_split = 0, a_split2 = 0, W = 1, n_main = 0;
    int my_start[2 * kTcMaxWaves] = {0, 0, 0, 0, 0, 0}, my_cnt[2 * kTcMaxWaves] = {0, 0, 0, 0, 0, 0},
        my_trim[2 * kTcMaxWaves] = {0, 0, 0, 0, 0, 0};
    // 2 W segments in time order: phase 1 of waves 0 .. W - 1, then phase 2 of waves 0 .. W - 1.
    // Contiguous units are consecutive k-pieces of one 128-row block, so a CTA accumulates them in
    // one TMEM accumulator and the epilogue runs once per run of k-pieces instead of once per
    // unit; only row blocks cut by a CTA boundary are reduced from two CTAs.
    auto unit_make = [&](int i) -> TcUnit {
        int seg = 0, j = i;
        while (seg < 2 * W - 1 && j >= my_cnt[seg]) { j -= my_cnt[seg]; ++seg; }
        const int start = my_start[seg], cnt = my_cnt[seg], trim = my_trim[seg];
        TcUnit t = tc_decode(groups, n_active, total1, start + j, sh.d, pl.n1);
        const int K = t.phase == 1 ? sh.d : groups[t.a].f;
        if (j == 0 && (trim & 1)) t.kt0 += kTcKT / 2;            // the CTA before this one has the first half
        if (j == cnt - 1 && (trim & 2)) t.kt1 -= kTcKT / 2;      // the next CTA has the second half
        t.seg = seg;
        t.first = (j == 0 || t.kt0 == 0) ? 1 : 0;
        t.last = (j == cnt - 1 || t.kt1 == (K + 63) / 64) ? 1 : 0;
        return t;
    };
    auto build_tables = [&](int tt, int tn, int bar_id) {
        n_active = ws.header[0];
        U = ws.header[2];
        const int ne = EARLY ? n_early : 0;
        // one round of global loads: the header above, the group table in its final form and the
        // slot arrays, whose sizes are known without the header
        for (int a = tt; a < G; a += tn) {
            const uint4 r0 = ws.gtab[2 * a], r1 = ws.gtab[2 * a + 1];
            if (a < n_active) {
                TcGroup gr;
                gr.group = (int)r0.x;
                // offloaded experts: from here on the group id of a routed expert is the device slot its
                // weights lie in (a slot index is below E as well, so shared groups stay recognisable)
                if (ws.slot_of && gr.group < sh.E) gr.group = __ldg(&ws.slot_of[gr.group]);
                gr.T = (int)r0.y;
                gr.off = (int)r0.z;
                gr.f = gr.group < sh.E ? sh.f : sh.f_sh;
                gr.mask = (unsigned long long)r1.x | ((unsigned long long)r1.y << 32);
                const int r = a < U ? a : U, s = a < U ? 0 : a - U;
                // (early start: the first projection of the early and the shared experts is in the pre-lot)
                gr.p1 = EARLY ? max(0, r - ne) * u1r : r * u1r + s * u1s;
                gr.p2 = r * u2r + s * u2s;
                // (the early experts must lead the final list in the order they were announced in)
                if (EARLY && a < ne && groups[a].group != gr.group) atomicExch(ws.status, ST_BAD_PLAN);
                groups[a] = gr;
            }
        }
        for (int i = tt; i < n_slots; i += tn) {
            s_slot_token[i] = ws.slot_token[i];
            s_slot_w[i] = ws.slot_w[i];
        }
        total1 = EARLY ? max(0, U - ne) * u1r : U * u1r + sh.n_sh * u1s;
        total2 = U * u2r + sh.n_sh * u2s;
        if (tt == 0) {
            // wave w starts at the first group whose first-projection units (pre-lot included) begin at
            // or after its share of all of them (in 16ths: pl.split[w - 1]; 16: no such wave)
            int sp = 0;
            for (int w = 0; w < 2; ++w) {
                if (pl.split[w] >= 16 || n_active < 2) sp = n_active;
                else {
                    if (sp < 1) sp = 1;
                    if (w == 1 && sp < n_active) ++sp;   // (a wave has at least one group)
                    while (sp < n_active - 1) {
                        const int r = sp < U ? sp : U, q = sp < U ? 0 : sp - U;
                        if ((long long)(r * u1r + q * u1s) * 16 >= (long long)(U * u1r + sh.n_sh * u1s) * pl.split[w]) break;
                        ++sp;
                    }
                    if (sp > n_active) sp = n_active;
                }
                s_split[w] = sp;
            }
        }
        asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(tn) : "memory");
        a_split = s_split[0];
        a_split2 = s_split[1];
        W = 1 + (a_split < n_active ? 1 : 0) + (a_split2 < n_active ? 1 : 0);
        {
            // first unit of every wave in both projections
            int b1[kTcMaxWaves + 1], b2[kTcMaxWaves + 1];
            b1[0] = 0; b2[0] = 0;
            b1[1] = a_split < n_active ? groups[a_split].p1 : total1;  b2[1] = a_split < n_active ? groups[a_split].p2 : total2;
            b1[2] = a_split2 < n_active ? groups[a_split2].p1 : total1; b2[2] = a_split2 < n_active ? groups[a_split2].p2 : total2;
            b1[W] = total1; b2[W] = total2;
            n_main = 0;
            for (int w = 0; w < W; ++w) share(b1[w], b1[w + 1] - b1[w], halves1, my_start[w], my_cnt[w], my_trim[w]);
            for (int w = 0; w < W; ++w)
                share(total1 + b2[w], b2[w + 1] - b2[w], halves2, my_start[W + w], my_cnt[W + w], my_trim[W + w]);
            for (int g = 0; g < 2 * W; ++g) n_main += my_cnt[g];
        }
        if (EARLY && n_pre + n_main > kTcMaxUnits) {  // (see above: left off by the host)
            if (tt == 0) atomicExch(ws.status, ST_BAD_PLAN);
            n_main = kTcMaxUnits - n_pre;
        }
        // decoded once: the single-thread roles below then read a unit from shared memory instead
        // of dividing
        for (int i = tt; i < n_main && n_pre + i < kTcMaxUnits; i += tn) {
            const TcUnit t = unit_make(i);
            s_units[n_pre + i] = t;
            s_umeta[n_pre + i] = tc_unit_meta(t);
        }
        asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(tn) : "memory");
    };
    if (!EARLY) {
        // programmatic dependent launch: the routing kernel in front of this grid must have
        // finished before its results are read; the next layer's routing kernel may be scheduled
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        tc_fence_before();
        build_tables(tid, (int)blockDim.x, 0);
        tc_fence_after();
    } else if (warp >= 7) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        build_tables(tid - 224, 128, 1);
        if (tid == 224) {
            s_tab[0] = n_main;
            s_tab[1] = n_active;
            mbar_arrive(&tab_bar);                    // (release: the tables are written)
        }
    }
    const uint32_t tmem_base = s_tmem;
    // What a role knows of the tables: everything at once, or (early start) after tab_bar.  The
    // roles keep their own copies (lim: units of this CTA known so far).
    auto tables_wait = [&](int &lim, int &split, int &split2, int &waves) -> bool {
        if (!mbar_wait(&tab_bar, 0)) { atomicExch(ws.status, ST_MBAR_TIMEOUT); return false; }
        lim = n_pre + s_tab[0];
        split = s_split[0];
        split2 = s_split[1];
        waves = 1 + (split < s_tab[1] ? 1 : 0) + (split2 < s_tab[1] ? 1 : 0);
        return true;
    };
    const int n_units0 = EARLY ? n_pre : n_main;      // units known when the roles start
    const int n_units = n_units0;                     // (the int4 roles: all of them)
    auto unit_at = [&](int i) -> TcUnit { return i < kTcMaxUnits ? s_units[i] : unit_make(i); };
    auto umeta_at = [&](int i) -> uint32_t { return i < kTcMaxUnits ? s_umeta[i] : tc_unit_meta(unit_make(i)); };

    if (warp == 0) {
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
            TcUnit pu = unit_at(0), tu = pu;
            int pkt = pu.kt0, tkt = pu.kt0;
            int s = 0, ta = 0;
            uint32_t ring_par = 1, t_par = 1;
            int ready_w = 0;
            unsigned idle = 0;
            bool alive = n_units > 0;

            while (alive && (pi < n_units || ti < n_units)) {
                bool progress = false;
                if (pi < n_units && mbar_test(&empty_bar[s], ring_par)) {

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
                    if (pkt >= pu.kt1 && ++pi < n_units) { pu = unit_at(pi); pkt = pu.kt0; }
                    progress = true;

                }
                if (ti < n_units) {
                    const int wv = tu.a >= a_split ? 1 : 0;
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
                        if (tkt >= tu.kt1 && ++ti < n_units) { tu = unit_at(ti); tkt = tu.kt0; }
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
                if (pl.kg == 2) {
                    // one copy per 8 slots for both k-tiles: [hi | lo][k-tile][8 rows]
                    for (int r = 0; r < tn / 2; r += 8) tma_load_4d(op + r * 512, am, 0, srow + r, kt, 0, &full_bar[s]);
                    return;
                }
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

            int lim = n_units0, a_split_p = a_split, a_split2_p = a_split2, w_p = W;
            bool tabs = !EARLY;
            for (int i = 0; alive; ++i) {
                if (i >= lim) {
                    // (early start: the pre-lot is on its way; the rest needs the tables)
                    if (tabs) break;
                    tabs = true;
                    if (!tables_wait(lim, a_split_p, a_split2_p, w_p)) { alive = false; break; }
                    if (i >= lim) break;
                }

                const TcUnit t = unit_at(i);
                const TcGroup &g = groups[t.a];
                const bool shared = g.group >= sh.E;
                const int e = shared ? g.group - sh.E : g.group;
                const CUtensorMap *wmap = &maps.m[(shared ? 3 : 0) + t.mat];
                const int rows_per_e = t.mat == 2 ? sh.d : g.f;
                const int row0 = e * rows_per_e + t.rb * 128;
                const int srow = shared ? g.off - n_routed : g.off;   // row in the routed / shared activation array
                const int wv = (t.a >= a_split_p ? 1 : 0) + (t.a >= a_split2_p ? 1 : 0);
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

                const int KGB = pl.kg;                     // k-tiles per stage (1 or 2)
                for (int kt = t.kt0; kt < t.kt1 && alive; kt += KGB, ++it, tc_ring_next(s, ring_par, S)) {
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
                    if (KGB == 2) {
                        // both k-tiles of the stage in one weight copy (a k-tile past the end of the
                        // contraction reads as zero) and one token copy (phase 2: one per 8 slots)
                        const uint32_t op_bytes = t.phase == 1 ? (pl.x_bytes ? 0u : 2u * (uint32_t)pl.tokb) : 2u * (uint32_t)t.n * 128u;
                        mbar_expect_tx(&full_bar[s], 2 * kTcWTile + op_bytes);
                        tma_load_3d_stream(stage, &maps.m[9 + (shared ? 3 : 0) + t.mat], 0, row0, kt, &full_bar[s], wpolicy);
                        if (t.phase == 1) {
                            if (!pl.x_bytes) tma_load_3d(stage + pl.tok_off, &maps.m[6], 0, 0, kt, &full_bar[s]);
                        } else if (ready) {
                            load_tokens2(s, kt, srow, shared, t.n);
                        } else {
                            pend_stage[pend_n] = s; pend_kt[pend_n] = kt; pend_row[pend_n] = srow;
                            pend_shared[pend_n] = shared; pend_tn[pend_n] = t.n;
                            pend_wave = wv;
                            ++pend_n;
                        }
                        continue;
                    }
                    const uint32_t op_bytes = t.phase == 1 ? (pl.x_bytes ? 0u : (uint32_t)t.n * 128u) : (uint32_t)t.n * 128u;
                    mbar_expect_tx(&full_bar[s], kTcWTile + op_bytes);
                    tma_load_2d_stream(stage, wmap, kt * 64, row0, &full_bar[s], wpolicy);
                    if (t.phase == 1) {
                        if (!pl.x_bytes)
                            for (int r = 0; r < t.n; r += pl.rows1)
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
            unsigned it = 0, ui = 0, run = 0;
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
                    for (int r = 0; r < pl.n1; r += pl.rows1)
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
            const uint32_t hi_p2k = (uint32_t)(tc_smem_desc_sbo(ring, 2048u) >> 32);     // bf16, two k-tiles per stage
            const unsigned nbm = (unsigned)pl.n_acc - 1u, nbs = (unsigned)__ffs(pl.n_acc) - 1u;   // accumulator buffers: mask, log2
            const uint32_t ring_lo = (uint32_t)tc_smem_desc(ring) + koff, xres_lo = (uint32_t)tc_smem_desc(xres) + koff;
            const uint32_t tok_lo = (uint32_t)tc_smem_desc(tokring) + koff;
            const uint32_t a_tmem0 = tmem_base + (uint32_t)kTcQ4ACol + 4u * koff;     // 8 columns per K-step

            if (Q4) {
                // int4: a unit is one stage; everything this thread needs of it is one word
                uint32_t d_tmem = tmem_base + (uint32_t)(half * 2 * pl.n1), buf = 0, run_par = 1;
                const uint32_t tok_slot = (uint32_t)kTcQ4KG * ((uint32_t)pl.tokb >> 4), tok_step1 = (uint32_t)pl.tokb >> 4;
                for (; (int)ui < n_units; ++ui) {
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
            for (int lim = n_units0, tabs = EARLY ? 0 : 1; alive; ++ui) {
                if ((int)ui >= lim) {
                    int sp_, sp2_, w_;
                    if (tabs) break;
                    tabs = 1;
                    if (!tables_wait(lim, sp_, sp2_, w_) || (int)ui >= lim) break;
                }
                const TcUnit t = unit_at((int)ui);
                const int buf = run & nbm;
                if (t.first) {

                    if (!mbar_wait(&acc_empty[buf], ((run >> nbs) & 1u) ^ 1u)) {
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
                const int KGB = pl.kg;
                for (int kt = t.kt0; kt < t.kt1; kt += KGB, ++it, tc_ring_next(s, ring_par, S)) {

                    if (!mbar_wait(&full_bar[s], ring_par)) {
                        atomicExch(ws.status, ST_MBAR_TIMEOUT);
                        alive = false;
                        break;
                    }

                    tc_fence_after();

                    if (KGB == 2) {
                        // two weight k-tiles 16 KiB apart; their token tiles tokb apart (phase 1) or, per
                        // 8 slots, [hi | lo][k-tile][8 rows]: 8-row groups 2 KiB apart, k-tiles 1 KiB
                        const uint32_t a_lo = ring_lo + (uint32_t)s * ((uint32_t)pl.stage_bytes >> 4);
                        const bool p2 = t.phase == 2, xr = !p2 && pl.x_bytes;       // (resident hidden-state tiles: n1 rows each)
                        const uint32_t b0 = xr ? xres_lo + (uint32_t)kt * ((uint32_t)pl.n1 * 8u) : a_lo + ((uint32_t)pl.tok_off >> 4);
                        const uint32_t b_step = p2 ? 64u : (xr ? (uint32_t)pl.n1 * 8u : ((uint32_t)pl.tokb >> 4)), b_hi = p2 ? hi_p2k : hi_std;
#pragma unroll
                        for (uint32_t g = 0; g < 2; ++g)
                            for (uint32_t k = 0; k < ks; ++k) {
                                tc_mma_bf16_parts(d_tmem, a_lo + g * (kTcWTile >> 4) + 2 * k, hi_std, b0 + g * b_step + 2 * k, b_hi, idesc, acc);
                                acc = 1;
                            }
                    } else {
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
                    ++run;
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
            for (int ui = 0; ui < n_units && alive; ++ui, tc_ring_next(s, ring_par, S), tc_ring_next(ta, a_par, pl.a_stages)) {

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
                // all packed chunks of this thread first: the stores to tensor memory below order
                // memory accesses, so a load behind one of them would wait for it
                uint4 pks[CP];
#pragma unroll
                for (int qi = 0; qi < CP; ++qi) {
                    // the packed rows are swizzled over their own width by the TMA copy
                    const int sw = KG == 4 ? (r & 7) : (KG == 2 ? ((r >> 1) & 3) : ((r >> 2) & 1));
                    pks[qi] = *reinterpret_cast<const uint4 *>(prow + (((h * CP + qi) ^ sw) * 16));
                }
#pragma unroll
                for (int qi = 0; qi < CP; ++qi) {
                    const int q = h * CP + qi;                         // chunk of 32 weights inside the stage
                    const uint4 pk = pks[qi];
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
        long long el_b[kTcMaxWaves + 1];             // first element of every wave's activations
        el_b[0] = 0;
        el_b[1] = a_split < n_active ? (long long)act_offset(groups[a_split].off, n_routed, sh.f, sh.f_sh) : n_el;
        el_b[2] = a_split2 < n_active ? (long long)act_offset(groups[a_split2].off, n_routed, sh.f, sh.f_sh) : n_el;
        el_b[W] = n_el;

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
            // (act_offset(slot) + row): this CTA converts a contiguous slice of the wave's range,
            // four elements per thread and step
            const long long w_lo = el_b[w], w_hi = el_b[w + 1];
            const long long n4 = (w_hi - w_lo) >> 2;
            const long long lo4 = n4 * blockIdx.x / gridDim.x, hi4 = n4 * (blockIdx.x + 1) / gridDim.x;
            // eight loads in flight per thread (a slice is up to 13 passes of the 96 threads at 64 tokens:
            // one pass at a time was 1 us of memory latency each, on the hand-over's critical path)
            for (long long q0 = lo4 + et; q0 < hi4; q0 += 96 * 4) {
                float4 gv[4], uv[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const long long q = q0 + 96 * u, i = w_lo + 4 * q;
                    if (q < hi4) {
                        gv[u] = __ldcg(reinterpret_cast<const float4 *>(p.pre + i));
                        uv[u] = __ldcg(reinterpret_cast<const float4 *>(p.pre + n_el + i));
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const long long q = q0 + 96 * u, i = w_lo + 4 * q;
                    if (q >= hi4) continue;
                    const float a0 = silu_mul(gv[u].x, uv[u].x), a1 = silu_mul(gv[u].y, uv[u].y), a2 = silu_mul(gv[u].z, uv[u].z),
                                a3 = silu_mul(gv[u].w, uv[u].w);
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
        unsigned ui = 0, run = 0;
        uint32_t ep_phase = 0;
        const int n_routed = p.B * sh.k;
        bool alive = true;

        // ---- hand-over between the projections, per wave (see the header comment)
        const int n_routed_el = n_routed;   // (alias used below)
        (void)n_routed_el;
        const long long n_el = (long long)n_routed * sh.f + (long long)sh.n_sh * p.B * sh.f_sh;
        int next_arrive = 0;
        int lim = n_units0, a_split_e = a_split, a_split2_e = a_split2, w_e = W;
        bool tabs = !EARLY;
        const unsigned nbm = (unsigned)pl.n_acc - 1u, nbs = (unsigned)__ffs(pl.n_acc) - 1u;
        (void)a_split_e; (void)a_split2_e;
        auto wave_arrive = [&](int w) -> bool {
            // this CTA's phase-1 reductions of wave w are issued: hand over to the converter warps,
            // whose first thread orders them (fence) before it arrives on the grid-wide counter, so
            // that no epilogue thread stalls on a fence
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&conv_go[w]);

            }
            return true;
        };
        // called before every unit (and once at the end): hand a wave over once this CTA's phase-1
        // units of it are all done
        auto service = [&](int upcoming_seg) -> bool {
            // (segment w is phase 1 of wave w: it is done once a later segment comes up)
            while (next_arrive < w_e && upcoming_seg > next_arrive) {
                if (!wave_arrive(next_arrive)) return false;
                ++next_arrive;
            }
            return true;
        };
        {
            for (; alive; ++ui) {
                if ((int)ui >= lim) {
                    if (tabs) break;
                    tabs = true;
                    if (!tables_wait(lim, a_split_e, a_split2_e, w_e)) { alive = false; break; }
                    if ((int)ui >= lim) break;
                }
                const TcUnit t = unit_at((int)ui);
                if (!service(t.seg)) { alive = false; break; }
                if (!t.last) continue;                 // the run's accumulator is read after its last unit
                if (!tabs && t.a < GP) {
                    // an early routed expert of the pre-lot: its tokens and slots come with the tables
                    tabs = true;
                    if (!tables_wait(lim, a_split_e, a_split2_e, w_e)) { alive = false; break; }
                }
                const TcGroup &g = groups[t.a];
                const int buf = run & nbm;

                if (!mbar_wait(&acc_full[buf], (run >> nbs) & 1u)) {
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
                ++run;

            }
            if (alive && !service(2 * kTcMaxWaves)) alive = false;
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
