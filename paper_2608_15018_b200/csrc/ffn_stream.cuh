// Streaming expert kernel (kernel plan 2): one persistent CTA per SM reads every
// selected expert's weights from HBM exactly once through a ring of TMA bulk copies
// and contracts them with the tokens bucketed to that expert on the tensor cores.
//
// Work is cut into units of equal cost, taken round-robin by the CTAs:
//   phase 1 unit: 8 gate rows + 8 up rows of one expert (all of K = d)
//                 -> a[slot][j] = silu(g) * u, stored as bf16 hi + lo parts
//   phase 2 unit: 32 down rows of one expert, one K-slice of f
//                 -> y[token][r] += p * (W_d[r] . a[slot])        (red.add, fp32)
// All phase-1 units precede all phase-2 units; a phase-2 unit of an expert waits on a
// counter of that expert's finished phase-1 units (bounded wait).
//
// Inside a CTA one producer warp issues the copies (one cp.async.bulk per weight row
// chunk and per token row chunk, completing on an mbarrier) and eight consumer warps
// split each staged chunk along K.  The contraction is mma.sync m16n8k16 with the
// tokens as the M operand and eight weight rows as the N operand; the K index inside
// every 32-wide step is permuted identically for both operands so that each lane feeds
// the tensor core straight from one 128-bit shared-memory load per row.
#pragma once

#include "common.cuh"

namespace s2moe {

constexpr int kStConsumerWarps = 8;
constexpr int kStThreads = (kStConsumerWarps + 1) * 32;
constexpr int kStStages = 5;
constexpr int kStRegion = 18432;                       // bytes per operand / weight region of a slot
constexpr int kStSlotBytes = 2 * kStRegion;
constexpr int kStScratchBytes = 16384;
constexpr int kStMaxGroups = kMaxExperts + kMaxShared;
constexpr size_t kStSmemBytes = (size_t)kStStages * kStSlotBytes + kStScratchBytes;
constexpr unsigned kStSpinLimit = 1u << 22;            // bounded waits (each poll ~ 50-100 ns)

struct StageDesc {
    int unit, chunk, nchunks, group_slot;   // group_slot: index into the active list
    int phase, tile, T, off;                // tokens of the group, first slot
    int klen, pitch_w, pitch_o, tpad8;      // this chunk's K length, row pitches, padded tokens
    int f_g, k_begin, group, pad_;
};

struct StreamArgs {
    Shape sh;
    LayerPtrs lp;
    Workspace ws;
    const void *hidden;
    float *y;
    __nv_bfloat16 *act_hi, *act_lo;
};

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
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
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
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Barrier among the consumer warps built on an mbarrier so that the wait is bounded
// (a hardware bar.sync would hang for ever if a warp had left after a time-out).
// `phase` is the caller's running parity bit.  Returns false when it gave up.
__device__ __forceinline__ bool consumer_bar(uint64_t *bar, uint32_t &phase, int lane)
{
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    const bool ok = mbar_wait(bar, phase);
    phase ^= 1u;
    return ok;
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

// row pitch in shared memory: consecutive rows must differ by 64 bytes modulo 128 so
// that the 128-bit loads of a quarter warp (two rows x 64 bytes) hit distinct banks
__host__ __device__ __forceinline__ int st_pitch(int chunk_bytes)
{
    return (chunk_bytes % 128 == 64) ? chunk_bytes : chunk_bytes + 64;
}

// K elements staged per chunk for a group with tpad8 padded tokens
__host__ __device__ __forceinline__ int st_kc(int phase, int tpad8)
{
    const int rows_w = phase == 1 ? 16 : 32;
    const int rows_o = phase == 1 ? tpad8 : 2 * tpad8;
    int kc = phase == 1 ? 512 : 256;
    while (kc > 32 && (rows_w * st_pitch(kc * 2) > kStRegion || rows_o * st_pitch(kc * 2) > kStRegion)) kc >>= 1;
    return kc;
}

// number of K-slices of a phase-2 unit so that a unit holds at most 64 KiB of weights
__host__ __device__ __forceinline__ int st_nks2(int f_g)
{
    const int n = (32 * f_g * 2 + 65535) / 65536;
    return n < 1 ? 1 : n;
}
__host__ __device__ __forceinline__ int st_kslice2(int f_g) { return ((f_g / 32 + st_nks2(f_g) - 1) / st_nks2(f_g)) * 32; }

__device__ __forceinline__ int upper_group(const int *pfx, int n, int u)
{
    int lo = 0, hi = n;                 // largest a with pfx[a] <= u
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pfx[mid] <= u) lo = mid; else hi = mid;
    }
    return lo;
}

// ---- the kernel -----------------------------------------------------------------

template <int MT, int PHASE>
__device__ __forceinline__ bool consume_unit(const StreamArgs &p, uint8_t *slots, float *scratch, uint64_t *full_bar,
                                             uint64_t *empty_bar, const StageDesc *desc, unsigned &it, int warp,
                                             int lane, int ctid, uint64_t *cbar, uint32_t &cphase)
{
    constexpr int NT = PHASE == 1 ? 2 : 4;
    const int g = lane >> 2, t = lane & 3;
    float acc[MT][NT][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[m][n][q] = 0.f;

    StageDesc d;
    while (true) {
        const int slot = it % kStStages;
        const uint32_t parity = (it / kStStages) & 1u;
        if (!mbar_wait(&full_bar[slot], parity)) return false;
        d = desc[slot];
        const uint8_t *wreg = slots + (size_t)slot * kStSlotBytes;
        const uint8_t *oreg = wreg + kStRegion;
        const int nsteps = d.klen >> 5;
        for (int s = warp; s < nsteps; s += kStConsumerWarps) {
            const int boff = s * 64 + t * 16;
            uint4 xa[MT], xb[MT], la[MT], lb[MT];
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const int r0 = m * 16 + g, r1 = r0 + 8;
                xa[m] = *reinterpret_cast<const uint4 *>(oreg + (size_t)r0 * d.pitch_o + boff);
                xb[m] = r1 < d.tpad8 ? *reinterpret_cast<const uint4 *>(oreg + (size_t)r1 * d.pitch_o + boff)
                                     : make_uint4(0, 0, 0, 0);
                if (PHASE == 2) {
                    la[m] = *reinterpret_cast<const uint4 *>(oreg + (size_t)(d.tpad8 + r0) * d.pitch_o + boff);
                    lb[m] = r1 < d.tpad8
                                ? *reinterpret_cast<const uint4 *>(oreg + (size_t)(d.tpad8 + r1) * d.pitch_o + boff)
                                : make_uint4(0, 0, 0, 0);
                }
            }
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                const uint4 w = *reinterpret_cast<const uint4 *>(wreg + (size_t)(n * 8 + g) * d.pitch_w + boff);
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    mma_bf16(acc[m][n], xa[m].x, xb[m].x, xa[m].y, xb[m].y, w.x, w.y);
                    mma_bf16(acc[m][n], xa[m].z, xb[m].z, xa[m].w, xb[m].w, w.z, w.w);
                    if (PHASE == 2) {
                        mma_bf16(acc[m][n], la[m].x, lb[m].x, la[m].y, lb[m].y, w.x, w.y);
                        mma_bf16(acc[m][n], la[m].z, lb[m].z, la[m].w, lb[m].w, w.z, w.w);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[slot]);
        ++it;
        if (d.chunk == d.nchunks - 1) break;
    }

    // cross-warp reduction and epilogue, one m-tile (16 tokens) per round
    constexpr int COLS = NT * 8;
    const int n_routed = p.ws.header[3] * p.sh.k;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        float *mine = scratch + (size_t)warp * 16 * COLS;
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            *reinterpret_cast<float2 *>(&mine[g * COLS + n * 8 + 2 * t]) = make_float2(acc[m][n][0], acc[m][n][1]);
            *reinterpret_cast<float2 *>(&mine[(g + 8) * COLS + n * 8 + 2 * t]) =
                make_float2(acc[m][n][2], acc[m][n][3]);
        }
        if (!consumer_bar(cbar, cphase, lane)) return false;
        if (PHASE == 1) {
            if (ctid < 128) {
                const int tt = ctid >> 3, j = ctid & 7;
                const int ti = m * 16 + tt;
                float sg = 0.f, su = 0.f;
#pragma unroll
                for (int w = 0; w < kStConsumerWarps; ++w) {
                    sg += scratch[(size_t)w * 16 * COLS + tt * COLS + j];
                    su += scratch[(size_t)w * 16 * COLS + tt * COLS + 8 + j];
                }
                if (ti < d.T) {
                    const float a = silu_mul(sg, su);
                    const __nv_bfloat16 hi = __float2bfloat16_rn(a);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(a - __bfloat162float(hi));
                    const size_t o = act_offset(d.off + ti, n_routed, p.sh.f, p.sh.f_sh) + (size_t)d.tile * 8 + j;
                    p.act_hi[o] = hi;
                    p.act_lo[o] = lo;
                }
            }
            __threadfence();
            fence_proxy_async();
        } else {
            const int tt = ctid >> 4, c0 = (ctid & 15) * 2;
            const int ti = m * 16 + tt;
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int w = 0; w < kStConsumerWarps; ++w) {
                const float2 v = *reinterpret_cast<const float2 *>(&scratch[(size_t)w * 16 * COLS + tt * COLS + c0]);
                s0 += v.x;
                s1 += v.y;
            }
            if (ti < d.T) {
                const int slot = d.off + ti;
                const float pw = p.ws.slot_w[slot];
                float *dst = p.y + (size_t)p.ws.slot_token[slot] * p.sh.d + (size_t)d.tile * 32 + c0;
                atomicAdd(dst, pw * s0);
                atomicAdd(dst + 1, pw * s1);
            }
        }
        if (!consumer_bar(cbar, cphase, lane)) return false;
    }
    if (PHASE == 1 && ctid == 0) {
        atomicAdd(&p.ws.sync[d.group_slot], 1);
        atomicAdd(&p.ws.sync[kStMaxGroups], 1);
    }
    return true;
}

__global__ void __launch_bounds__(kStThreads, 1) ffn_stream_kernel(StreamArgs p)
{
    extern __shared__ __align__(128) uint8_t st_smem[];
    __shared__ __align__(8) uint64_t full_bar[kStStages];
    __shared__ __align__(8) uint64_t empty_bar[kStStages];
    __shared__ __align__(8) uint64_t cbar;
    __shared__ StageDesc desc[kStStages];
    __shared__ int s_pfx1[kStMaxGroups + 1], s_pfx2[kStMaxGroups + 1];

    uint8_t *slots = st_smem;
    float *scratch = reinterpret_cast<float *>(st_smem + (size_t)kStStages * kStSlotBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Workspace &ws = p.ws;
    const int n_active = ws.header[0];
    const int total1 = ws.header[4], total2 = ws.header[5];
    const int total = total1 + total2;

    for (int i = tid; i <= n_active; i += blockDim.x) {
        s_pfx1[i] = ws.upfx1[i];
        s_pfx2[i] = ws.upfx2[i];
    }
    if (tid == 0) {
        for (int s = 0; s < kStStages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kStConsumerWarps);
        }
        mbar_init(&cbar, kStConsumerWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const Shape &sh = p.sh;
    if (warp == kStConsumerWarps) {
        // ------------------------------------------------------------ producer warp
        unsigned it = 0;
        bool all_ready = false, alive = true;
        for (int u = blockIdx.x; u < total && alive; u += gridDim.x) {
            StageDesc d;
            d.unit = u;
            d.phase = u < total1 ? 1 : 2;
            int ks = 0;
            if (d.phase == 1) {
                d.group_slot = upper_group(s_pfx1, n_active, u);
                d.tile = u - s_pfx1[d.group_slot];
            } else {
                const int v = u - total1;
                d.group_slot = upper_group(s_pfx2, n_active, v);
                d.tile = v - s_pfx2[d.group_slot];
            }
            d.group = ws.active[d.group_slot];
            d.T = ws.counts[d.group];
            d.off = ws.offsets[d.group];
            d.tpad8 = (d.T + 7) & ~7;
            const bool shared = d.group >= sh.E;
            d.f_g = shared ? sh.f_sh : sh.f;
            const int e = shared ? d.group - sh.E : d.group;
            const int kc = st_kc(d.phase, d.tpad8);
            int klen_unit;
            const uint8_t *wrow0, *wrow1 = nullptr;   // first row of the unit (gate / down), up rows
            size_t row_stride;
            if (d.phase == 1) {
                d.k_begin = 0;
                klen_unit = sh.d;
                row_stride = (size_t)sh.d * 2;
                const size_t r0 = ((size_t)e * d.f_g + (size_t)d.tile * 8) * row_stride;
                wrow0 = (const uint8_t *)(shared ? p.lp.sh_gate : p.lp.w_gate) + r0;
                wrow1 = (const uint8_t *)(shared ? p.lp.sh_up : p.lp.w_up) + r0;
            } else {
                const int nks = st_nks2(d.f_g), ksl = st_kslice2(d.f_g);
                ks = d.tile % nks;
                d.tile = d.tile / nks;
                d.k_begin = ks * ksl;
                klen_unit = min(ksl, d.f_g - d.k_begin);
                row_stride = (size_t)d.f_g * 2;
                wrow0 = (const uint8_t *)(shared ? p.lp.sh_down : p.lp.w_down) +
                        ((size_t)e * sh.d + (size_t)d.tile * 32) * row_stride;
                // wait until every phase-1 unit of this group has stored its activations
                if (!all_ready) {
                    int ok = 0;
                    if (lane == 0) {
                        const int need = s_pfx1[d.group_slot + 1] - s_pfx1[d.group_slot];
                        for (unsigned i = 0; i < (kStSpinLimit >> 2); ++i) {
                            if (ld_acquire(&ws.sync[kStMaxGroups]) >= total1) { ok = 2; break; }
                            if (ld_acquire(&ws.sync[d.group_slot]) >= need) { ok = 1; break; }
                            __nanosleep(64);
                        }
                        if (!ok) atomicExch(ws.status, ST_DEP_TIMEOUT);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { alive = false; break; }
                    if (ok == 2) all_ready = true;
                    fence_proxy_async();
                }
            }
            d.nchunks = (klen_unit + kc - 1) / kc;
            const int rows_w = d.phase == 1 ? 16 : 32;
            const size_t n_routed = (size_t)ws.header[3] * sh.k;
            for (int c = 0; c < d.nchunks; ++c) {
                const int slot = it % kStStages;
                const uint32_t parity = ((it / kStStages) & 1u) ^ 1u;
                int ok = 1;
                if (lane == 0) ok = mbar_wait(&empty_bar[slot], parity) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) {
                    if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                    alive = false;
                    break;
                }
                d.chunk = c;
                d.klen = min(kc, klen_unit - c * kc);
                const int cbytes = d.klen * 2;
                d.pitch_w = st_pitch(cbytes);
                d.pitch_o = d.pitch_w;
                uint8_t *wreg = slots + (size_t)slot * kStSlotBytes;
                uint8_t *oreg = wreg + kStRegion;
                const size_t kbyte = (size_t)(d.k_begin + c * kc) * 2;
                if (lane == 0) {
                    desc[slot] = d;
                    const uint32_t total_bytes = (uint32_t)(rows_w + (d.phase == 1 ? d.T : 2 * d.T)) * cbytes;
                    mbar_expect_tx(&full_bar[slot], total_bytes);
                }
                __syncwarp();
                for (int r = lane; r < rows_w; r += 32) {
                    const uint8_t *src;
                    if (d.phase == 1) src = (r < 8 ? wrow0 + (size_t)r * row_stride : wrow1 + (size_t)(r - 8) * row_stride);
                    else src = wrow0 + (size_t)r * row_stride;
                    bulk_g2s(wreg + (size_t)r * d.pitch_w, src + kbyte, cbytes, &full_bar[slot]);
                }
                if (d.phase == 1) {
                    for (int r = lane; r < d.T; r += 32) {
                        const int tok = ws.slot_token[d.off + r];
                        bulk_g2s(oreg + (size_t)r * d.pitch_o,
                                 (const uint8_t *)p.hidden + ((size_t)tok * sh.d) * 2 + kbyte, cbytes, &full_bar[slot]);
                    }
                } else {
                    for (int r = lane; r < 2 * d.T; r += 32) {
                        const int ti = r < d.T ? r : r - d.T;
                        const __nv_bfloat16 *base = r < d.T ? p.act_hi : p.act_lo;
                        const size_t o = act_offset(d.off + ti, (int)n_routed, sh.f, sh.f_sh);
                        const int srow = r < d.T ? ti : d.tpad8 + ti;
                        bulk_g2s(oreg + (size_t)srow * d.pitch_o, (const uint8_t *)(base + o) + kbyte, cbytes,
                                 &full_bar[slot]);
                    }
                }
                ++it;
            }
        }
        // let every copy that was issued land before the CTA may exit
        if (!alive && lane == 0) {
            for (int s = 0; s < kStStages; ++s) {
                // a slot whose full barrier is pending completes when its bytes arrive; bounded wait
                for (unsigned i = 0; i < (1u << 16); ++i)
                    if (mbar_try_wait(&full_bar[s], 0) || mbar_try_wait(&full_bar[s], 1)) break;
            }
        }
    } else {
        // ------------------------------------------------------------ consumer warps
        unsigned it = 0;
        uint32_t cphase = 0;
        const int ctid = tid;
        for (int u = blockIdx.x; u < total; u += gridDim.x) {
            const int slot = it % kStStages;
            const uint32_t parity = (it / kStStages) & 1u;
            if (!mbar_wait(&full_bar[slot], parity)) {
                if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                break;
            }
            const StageDesc d0 = desc[slot];
            const int mt = (d0.tpad8 + 15) >> 4;
            bool ok;
            if (d0.phase == 1) {
                if (mt == 1) ok = consume_unit<1, 1>(p, slots, scratch, full_bar, empty_bar, desc, it, warp, lane, ctid, &cbar, cphase);
                else if (mt == 2) ok = consume_unit<2, 1>(p, slots, scratch, full_bar, empty_bar, desc, it, warp, lane, ctid, &cbar, cphase);
                else if (mt == 3) ok = consume_unit<3, 1>(p, slots, scratch, full_bar, empty_bar, desc, it, warp, lane, ctid, &cbar, cphase);
                else ok = consume_unit<4, 1>(p, slots, scratch, full_bar, empty_bar, desc, it, warp, lane, ctid, &cbar, cphase);
            } else {
                if (mt == 1) ok = consume_unit<1, 2>(p, slots, scratch, full_bar, empty_bar, desc, it, warp, lane, ctid, &cbar, cphase);
                else if (mt == 2) ok = consume_unit<2, 2>(p, slots, scratch, full_bar, empty_bar, desc, it, warp, lane, ctid, &cbar, cphase);
                else if (mt == 3) ok = consume_unit<3, 2>(p, slots, scratch, full_bar, empty_bar, desc, it, warp, lane, ctid, &cbar, cphase);
                else ok = consume_unit<4, 2>(p, slots, scratch, full_bar, empty_bar, desc, it, warp, lane, ctid, &cbar, cphase);
            }
            if (!ok) {
                if (lane == 0) atomicExch(ws.status, ST_MBAR_TIMEOUT);
                break;
            }
        }
    }
}

}  // namespace s2moe
