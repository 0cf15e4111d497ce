// The hand-off kernel of hg_logits.cuh with its contraction on the fifth-generation tensor cores (sm_100a):
//     O^T [D x heads] += V^T [D x tokens] . P^T [tokens x heads]
// issued as tcgen05.mma by ONE thread, both operands read from shared memory through matrix descriptors, the
// accumulator in tensor memory.  This contraction suits the asynchronous tensor core well: the chunk maximum is known
// before the first product (the logits come from the host), so the accumulator is never rescaled and nothing but the
// final read-out has to leave tensor memory; and the V tile, as the TMA tensor load leaves it (64 token rows of 128
// bytes per 64-component half, 128-byte swizzled), IS the canonical "M-major" A operand - M = 64 components, K = tokens
// - so no warp ever touches a V element.  The warps' work is the logits: warp h turns head h's logits of the chunk
// into m, l and P, and stores P (hi + lo 16-bit terms) as the K-major B operand [8 heads x 16 tokens] of every
// 16-token step.  Then warp 0 alone drives the stream: it waits for a tile, lane 0 issues the tile's MMAs (per step
// and half: hi and lo term) and commits them to the tile's "empty" barrier, and refills the ring; the other warps
// wait for the chunk's last commit, read the accumulator (tcgen05.ld) and write the partial.
//
// Grid (chunk, KV head, sequence), 256 threads, 32 columns of tensor memory per CTA (8 per 64-component half are used).
// Every wait is bounded; tensor memory is freed on every path.
#pragma once

#include "hg_logits.cuh"

namespace hg {

// ---- tensor-memory and tcgen05 primitives ------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {          // one whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {       // the warp that allocated
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// The barrier gets one arrival once every tcgen05.mma this thread has issued so far has completed.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// D (tensor memory, fp32) (+)= A (shared memory) . B (shared memory), 16-bit inputs; one thread.
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// 32 lanes x 8 consecutive 32-bit columns: thread t of the warp gets lane (base lane + t), columns c .. c + 7.
__device__ __forceinline__ void tmem_ld_32x8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: start address, leading and stride byte offsets (all in 16-byte units),
// descriptor version 1, swizzle mode (0: none, 2: 128-byte).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle) {
    return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | ((uint64_t)swizzle << 61);
}

constexpr uint32_t LGTC_TMEM_COLS = 32;

template <int D>
constexpr size_t logits_tc_smem_bytes(int chunk) {
    return 1024 + (size_t)lg_stages<D>() * LG_TILE * D * 2 + (size_t)((chunk + LG_TILE - 1) / LG_TILE * LG_TILE / 16) * 512;
}

template <int D, bool BF16>
__global__ void __launch_bounds__(LG_THREADS, LG_MIN_CTAS) logits_partial_tc_kernel(const __grid_constant__ CUtensorMap tmV, const LogitsParams p) {
    constexpr int TILE_BYTES = LG_TILE * D * 2;
    constexpr int HALVES = D / 64;                    // 64-component halves of a V row: one M = 64 product each
    constexpr int HALF_BYTES = LG_TILE * 128;
    constexpr int LG_STAGES = lg_stages<D>();
    constexpr int STEPS = LG_TILE / 16;               // 16-token steps (K of one MMA) per tile
    constexpr float LOG2E = 1.4426950408889634f;
    const float NEG_INF = __int_as_float(0xff800000);
    // instruction descriptor: fp32 accumulator, A and B of the 16-bit type, A M-major (a V row's components are
    // contiguous), B K-major, N = 8, M = 64
    constexpr uint32_t FMT = BF16 ? 1u : 0u;
    constexpr uint32_t IDESC = (1u << 4) | (FMT << 7) | (FMT << 10) | (1u << 15) | ((8u >> 3) << 17) | ((64u >> 4) << 24);

    extern __shared__ uint8_t lg_raw[];
    __shared__ uint64_t full[LG_STAGES], empty[LG_STAGES], done;
    __shared__ float s_m[8], s_l[8];
    __shared__ int abort_flag_s;
    __shared__ uint32_t tmem_slot;
    const uint32_t tile0 = (smem_u32(lg_raw) + 1023u) & ~1023u;
    uint8_t* const tile0_ptr = lg_raw + (tile0 - smem_u32(lg_raw));
    const uint32_t p0 = tile0 + LG_STAGES * TILE_BYTES;               // P: per 16-token step 256 bytes of hi terms, 256 of lo
    uint8_t* const p0_ptr = tile0_ptr + LG_STAGES * TILE_BYTES;

    const int c = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = min(max(p.n_sel[b], 0), p.K);
    const int t0 = c * p.chunk, t1 = min(t0 + p.chunk, n);
    const int nt = max(t1 - t0, 0);                                   // slots of this chunk in use
    const int ntiles = (nt + LG_TILE - 1) / LG_TILE, nsteps = ntiles * STEPS;
    const int head_blocks = (p.G + 7) / 8;
    const int total = ntiles * head_blocks;                           // tiles this CTA streams, head block after head block
    const int row_base = (b * p.Hkv + g) * p.K + t0;                  // first V row of the chunk in the [B*Hkv*K][D] view
    volatile int* abort_flag = &abort_flag_s;

    if (tid == 0) {
        prefetch_tensormap(&tmV);
        for (int s = 0; s < LG_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(&done, 1);
        abort_flag_s = 0;
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(&tmem_slot, LGTC_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

    auto issue = [&](int i) {                                          // tile i of the CTA's sequence into slot i % LG_STAGES
        const int s = i % LG_STAGES;
        mbar_arrive_expect_tx(&full[s], TILE_BYTES);
        tma_load_3d(tile0_ptr + (size_t)s * TILE_BYTES, &tmV, &full[s], 0, row_base + (i % ntiles) * LG_TILE, 0);
    };
    int issued = 0;                                                    // (thread 0) tiles requested so far
    if (tid == 0)
        for (; issued < total && issued < LG_STAGES; ++issued) issue(issued);

    int it = 0;                                                        // (warp 0) tiles handed to the tensor core so far
    bool ok = true;
    for (int hb = 0; hb < head_blocks && ok; ++hb) {
        const int h0 = g * p.G + hb * 8, nh = min(8, p.G - hb * 8);
        // ---- warp h: head h's logits -> m, l and the B operands --------------------------------------------------
        // (the barrier: the previous block's accumulator has been read, its m and l written out)
        if (hb > 0) __syncthreads();
        {
            // a lane owns token pairs (2u, 2u + 1), u = lane + 32 i: coalesced 8-byte loads; the chunk's first 256 slots
            // stay in registers between the maximum and the weights, the rest is read twice
            float mx = NEG_INF;
            const bool live = warp < nh;
            const float* row = p.logits + ((size_t)b * p.Hq + h0 + (live ? warp : 0)) * p.K + t0;
            const bool vec_ok = ((reinterpret_cast<uintptr_t>(row) & 7u) == 0);
            auto pair_at = [&](int u) -> float2 {
                float2 v = make_float2(NEG_INF, NEG_INF);
                if (live && 2 * u < nt) {
                    if (vec_ok && 2 * u + 1 < nt) v = *reinterpret_cast<const float2*>(row + 2 * u);
                    else { v.x = row[2 * u]; if (2 * u + 1 < nt) v.y = row[2 * u + 1]; }
                }
                return v;
            };
            float2 first[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) first[j] = pair_at(lane + 32 * j);
#pragma unroll
            for (int j = 0; j < 4; ++j) mx = fmaxf(mx, fmaxf(first[j].x, first[j].y));
            for (int u0 = 128; 2 * u0 < nt; u0 += 128) {
                float2 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) v[j] = pair_at(u0 + lane + 32 * j);
#pragma unroll
                for (int j = 0; j < 4; ++j) mx = fmaxf(mx, fmaxf(v[j].x, v[j].y));
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float msafe = (mx == NEG_INF) ? 0.f : mx;
            float sum = 0.f;
            for (int u0 = 0; 2 * u0 < nsteps * 16; u0 += 128) {        // pair index u: step u / 8, position u % 8 in it
                float2 sv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) sv[j] = u0 == 0 ? first[j] : pair_at(u0 + lane + 32 * j);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int u = u0 + lane + 32 * j;
                    if (2 * u >= nsteps * 16) break;
                    const float w0 = live ? fast_exp2((sv[j].x - msafe) * LOG2E) : 0.f;   // e^{-inf} = 0 for unused slots
                    const float w1 = live ? fast_exp2((sv[j].y - msafe) * LOG2E) : 0.f;
                    sum += w0 + w1;
                    const uint32_t hi = pack2<BF16>(w0, w1);
                    const float2 f = unpack2<BF16>(hi);
                    const uint32_t lo = pack2<BF16>(w0 - f.x, w1 - f.y);
                    // B operand of step kt, K-major without swizzle: two 128-byte core matrices (tokens 0-7, 8-15 of the
                    // step), each 8 head rows of 16 bytes; this lane's pair is tokens 2 w8, 2 w8 + 1 of head `warp`
                    const int kt = u >> 3, w8 = u & 7;
                    uint8_t* dst = p0_ptr + (size_t)kt * 512 + (w8 >> 2) * 128 + warp * 16 + (w8 & 3) * 4;
                    *reinterpret_cast<uint32_t*>(dst) = hi;
                    *reinterpret_cast<uint32_t*>(dst + 256) = lo;
                }
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0 && live) { s_m[warp] = mx; s_l[warp] = sum; }
        }
        fence_proxy_async();                  // the tensor core reads P through the asynchronous proxy
        __syncthreads();

        // ---- warp 0: the chunk's tiles through the tensor core --------------------------------------------------
        if (warp == 0) {
            tc_fence_after_sync();
            for (int ti = 0; ti < ntiles; ++ti, ++it) {
                if (lane == 0 && it >= 1 && it - 1 + LG_STAGES < total) {
                    // the slot of the tile before this one is free once its products are done: refill it
                    if (mbar_wait(&empty[(it - 1) % LG_STAGES], (uint32_t)((it - 1) / LG_STAGES) & 1u, abort_flag)) {
                        issue(it - 1 + LG_STAGES);
                        ++issued;
                    }
                }
                const int s = it % LG_STAGES;
                ok = warp_wait(&full[s], (uint32_t)(it / LG_STAGES) & 1u, abort_flag);
                if (!ok) break;
                const uint32_t vbase = tile0 + s * TILE_BYTES;
                if ((ti + 1) * LG_TILE > nt) {
                    // rows past the chunk's last slot hold whatever lies behind it (other slots, NaN patterns): clear them
                    // (whole 128-byte rows, so the swizzle does not matter), and let the tensor core see the zeros
                    const int first_bad = nt - ti * LG_TILE;
                    for (int u = lane + first_bad * (HALVES * 8); u < LG_TILE * HALVES * 8; u += 32) {
                        const int r = u / (HALVES * 8), q = u % (HALVES * 8);
                        sts128_zero(vbase + (q >> 3) * HALF_BYTES + r * 128u + ((q & 7) << 4));
                    }
                    fence_proxy_async();
                }
                __syncwarp();
                if (lane == 0) {
                    tc_fence_after_sync();
#pragma unroll
                    for (int k4 = 0; k4 < STEPS; ++k4) {
                        const uint32_t pb = p0 + (uint32_t)(ti * STEPS + k4) * 512u;
                        const uint64_t b_hi = tc_smem_desc(pb, 128u, 256u, 0u), b_lo = tc_smem_desc(pb + 256u, 128u, 256u, 0u);
#pragma unroll
                        for (int h = 0; h < HALVES; ++h) {
                            // A: 64 components x 16 tokens of half h: token rows of 128 bytes, 8-row swizzle atoms 1024 bytes apart
                            const uint64_t a = tc_smem_desc(vbase + h * HALF_BYTES + k4 * (16 * 128), (uint32_t)HALF_BYTES, 1024u, 2u);
                            tc_mma_f16(tmem + h * 8, a, b_hi, IDESC, (ti | k4) != 0 ? 1u : 0u);
                            tc_mma_f16(tmem + h * 8, a, b_lo, IDESC, 1u);
                        }
                    }
                    tc_commit(&empty[s]);                              // the slot is free when these products are done
                    if (ti == ntiles - 1) tc_commit(&done);            // ... and so is the chunk
                }
                __syncwarp();
            }
        }
        // ---- all warps: the accumulator is complete; warps 0-3 read their 32 lanes of it -------------------------
        if (ntiles > 0) {
            ok = warp_wait(&done, (uint32_t)hb & 1u, abort_flag) && ok;
        }
        ok = __syncthreads_and(ok ? 1 : 0) != 0;          // the outcome is made uniform: all warps go on or none does
        if (!ok) break;
        if (warp < 4) {
            tc_fence_after_sync();
            // M = 64 products keep row 16 j + i of a half in lane 32 j + i (i < 16): lanes 16-31 of each quarter are unused
            uint32_t r[HALVES][8];
#pragma unroll
            for (int h = 0; h < HALVES; ++h) {
                if (ntiles > 0) tmem_ld_32x8(tmem + ((uint32_t)(warp * 32) << 16) + h * 8, r[h]);
                else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) r[h][j] = 0u;
                }
            }
            tmem_ld_wait();
            if (lane < 16) {
#pragma unroll
                for (int h = 0; h < HALVES; ++h) {
                    const int d = h * 64 + warp * 16 + lane;
#pragma unroll
                    for (int hh = 0; hh < 8; ++hh)
                        if (hh < nh) p.o_part[(((size_t)b * p.Hq + h0 + hh) * p.NC + c) * D + d] = __uint_as_float(r[h][hh]);
                }
            }
            if (warp == 0 && lane < nh) {
                const size_t slot = ((size_t)b * p.Hq + h0 + lane) * p.NC + c;
                p.m_part[slot] = s_m[lane];
                p.l_part[slot] = s_l[lane];
            }
            tc_fence_before_sync();
        }
    }
    __syncthreads();
    if (tid == 0 && *abort_flag) {
        // unwinding: copies into this CTA's shared memory may still be on their way
        for (int i = max(0, issued - LG_STAGES); i < issued; ++i) {
            int dummy = 0;
            mbar_wait(&full[i % LG_STAGES], (uint32_t)(i / LG_STAGES) & 1u, &dummy);
        }
        if (p.status) atomicOr(p.status, HG_DEV_WAIT_TIMEOUT);
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, LGTC_TMEM_COLS);
}

}  // namespace hg
