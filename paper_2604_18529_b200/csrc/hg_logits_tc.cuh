// The hand-off kernel of hg_logits.cuh with its contraction on the fifth-generation tensor cores (sm_100a):
//     O^T [D x heads] += V^T [D x tokens] . P^T [tokens x heads]
// issued as tcgen05.mma by ONE thread, both operands read from shared memory through matrix descriptors, the
// accumulator in tensor memory.  This contraction suits the asynchronous tensor core well: the chunk maximum is known
// before the first product (the logits come from the host), so the accumulator is never rescaled and nothing but the
// final read-out has to leave tensor memory; and the V tile, as the TMA tensor load leaves it (64 token rows of 128
// bytes per 64-component half, 128-byte swizzled), IS the canonical "M-major" A operand - M = the D components of a row, K = tokens
// - so no warp ever touches a V element.  That frees the warps for the one thing that used to stop the stream - the
// chunk's logits - and lets it run beside the stream instead of in front of it:
//
//   * persistent CTAs (two per SM, 320 threads) take work items (chunk, KV head, sequence, block of 8 heads) in turn;
//   * one thread of the loader warp keeps a ring of V tiles in flight ACROSS items;
//   * the tensor-core warp hands every landed tile to the tensor core (one product per 16-token step) and lets the
//     products' completion free the tile's slot (tcgen05.commit on the slot's "empty" barrier) and, after an item's
//     last tile, announce the item ("done");
//   * head warp h meanwhile turns head h's logits of the NEXT item into m, l and P, stored (hi + lo 16-bit terms)
//     as the K-major B operand [16 rows x 16 tokens] of every 16-token step; warps 0-3 then read the accumulator of
//     the item before the previous one out of tensor memory (tcgen05.ld) and write the partial.  P, the accumulator and their barriers
//     are double-buffered by item parity.
//
// One product per 16-token step: M = D, N = 16 (the 8 heads' hi terms and their 8 lo terms side by side; the read-out
// adds columns j and j + 8).  Every wait is bounded; tensor memory (32 columns per CTA, 16 per accumulator) is freed on
// every path.
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
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                   "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
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
constexpr int LGTC_HEAD_WARPS = 8;
constexpr int LGTC_LOAD_WARP = LGTC_HEAD_WARPS, LGTC_MMA_WARP = LGTC_HEAD_WARPS + 1;
constexpr int LGTC_THREADS = (LGTC_HEAD_WARPS + 2) * 32;   // eight head warps, the loader and the tensor-core warp
constexpr int LGTC_MAX_STAGES = 8;
constexpr int LGTC_CTAS_PER_SM = 2;     // (three, with rings of three tiles, measured the same at D = 128)
constexpr int LGTC_SMEM_BUDGET = 112 * 1024;               // dynamic shared memory of one of an SM's two CTAs

__host__ __device__ constexpr size_t lgtc_p_bytes(int chunk) { return (size_t)((chunk + LG_TILE - 1) / LG_TILE * LG_TILE / 16) * 512; }

// V tiles the ring of one CTA can hold beside the two P buffers (0: the chunk is too large for this kernel).
template <int D>
constexpr int lgtc_stages(int chunk) {
    const long long room = (long long)LGTC_SMEM_BUDGET - 1024 - 2 * (long long)lgtc_p_bytes(chunk);
    const long long n = room / (LG_TILE * D * 2);
    return n < 2 ? 0 : (n > LGTC_MAX_STAGES ? LGTC_MAX_STAGES : (int)n);
}
template <int D>
constexpr size_t logits_tc_smem_bytes(int chunk) {
    return 1024 + (size_t)lgtc_stages<D>(chunk) * LG_TILE * D * 2 + 2 * lgtc_p_bytes(chunk);
}

// One work item: chunk c of (sequence b, KV head g), block hb of up to 8 query heads.
struct LgItem {
    int b, g, c, hb;
    int nt;          // slots of the chunk in use (0: an empty partial)
    int row_base;    // first V row of the chunk in the [B * Hkv * K][D] view
};
constexpr int LGTC_NSEL_CACHE = 256;       // sequences whose slot counts are kept in shared memory
// (every role decodes every item of its CTA: the decode must not wait for global memory, and the item index is 32 bits
// wide - the host takes the other kernel for more than 2^31 items)
__device__ __forceinline__ LgItem lg_item(const LogitsParams& p, const int* s_nsel, uint32_t i) {
    LgItem it;
    it.hb = (int)(i % (uint32_t)p.head_blocks); i /= (uint32_t)p.head_blocks;
    it.c = (int)(i % (uint32_t)p.NC); i /= (uint32_t)p.NC;
    it.g = (int)(i % (uint32_t)p.Hkv);
    it.b = (int)(i / (uint32_t)p.Hkv);
    const int n = min(max(it.b < LGTC_NSEL_CACHE ? s_nsel[it.b] : p.n_sel[it.b], 0), p.K);
    const int t0 = it.c * p.chunk;
    it.nt = max(min(t0 + p.chunk, n) - t0, 0);
    it.row_base = (it.b * p.Hkv + it.g) * p.K + t0;
    return it;
}

template <int D, bool BF16>
__global__ void __launch_bounds__(LGTC_THREADS, LGTC_CTAS_PER_SM) logits_partial_tc_kernel(const __grid_constant__ CUtensorMap tmV, const LogitsParams p) {
    constexpr int TILE_BYTES = LG_TILE * D * 2;
    constexpr int HALVES = D / 64;                    // 64-component halves of a V row
    constexpr int HALF_BYTES = LG_TILE * 128;
    constexpr int STEPS = LG_TILE / 16;               // 16-token steps (K of one MMA) per tile
    constexpr float LOG2E = 1.4426950408889634f;
    const float NEG_INF = __int_as_float(0xff800000);
    // instruction descriptor: fp32 accumulator, A and B of the 16-bit type, A M-major (a V row's components are
    // contiguous), B K-major, M = D (all components of a V row in one product), N = 16: the 8 heads' hi terms and
    // their 8 lo terms side by side, so that one product per 16-token step does what would otherwise take four -
    // the columns j and j + 8 of the accumulator are added when it is read out
    constexpr uint32_t FMT = BF16 ? 1u : 0u;
    constexpr uint32_t IDESC = (1u << 4) | (FMT << 7) | (FMT << 10) | (1u << 15) | ((16u >> 3) << 17) | ((uint32_t)(D >> 4) << 24);
    constexpr uint32_t ACC_COLS = 16;

    extern __shared__ uint8_t lg_raw[];
    __shared__ uint64_t full[LGTC_MAX_STAGES], empty[LGTC_MAX_STAGES], p_ready[2], done[2], acc_free[2];
    __shared__ int abort_flag_s;
    __shared__ uint32_t tmem_slot;
    __shared__ int s_nsel[LGTC_NSEL_CACHE];
    const int S = p.stages;
    const uint32_t tile0 = (smem_u32(lg_raw) + 1023u) & ~1023u;
    uint8_t* const tile0_ptr = lg_raw + (tile0 - smem_u32(lg_raw));
    const uint32_t pbytes = (uint32_t)lgtc_p_bytes(p.chunk);
    const uint32_t p0 = tile0 + S * TILE_BYTES;                       // P[j]: per 16-token step 256 bytes of hi terms, 256 of lo
    uint8_t* const p0_ptr = tile0_ptr + (size_t)S * TILE_BYTES;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &abort_flag_s;

    if (tid == 0) {
        prefetch_tensormap(&tmV);
        for (int s = 0; s < S; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int j = 0; j < 2; ++j) { mbar_init(&p_ready[j], LGTC_HEAD_WARPS); mbar_init(&done[j], 1); mbar_init(&acc_free[j], 4); }
        abort_flag_s = 0;
        fence_barrier_init();
    }
    for (int bb = tid; bb < p.B && bb < LGTC_NSEL_CACHE; bb += LGTC_THREADS) s_nsel[bb] = p.n_sel[bb];
    if (warp == LGTC_MMA_WARP) {
        tmem_alloc(&tmem_slot, LGTC_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

    int issued = 0;                                                    // (loader) tiles requested so far
    if (warp == LGTC_LOAD_WARP) {
        // =============================== loader: one thread keeps the ring of V tiles full ===============================
        // (a tensor load and its barrier arming cost the issuing thread several hundred cycles, a product about a
        // hundred and fifty: one thread doing both for a 16 KB tile is slower than the tile's share of the memory
        // bandwidth, so the two are separate warps)
        if (lane == 0) {
            bool ok = true;
            for (uint32_t i = blockIdx.x; i < (uint32_t)p.items && ok; i += gridDim.x) {
                const LgItem cur = lg_item(p, s_nsel, i);
                const int ntiles = (cur.nt + LG_TILE - 1) / LG_TILE;
                for (int ti = 0; ti < ntiles; ++ti, ++issued) {
                    const int slot = issued % S;
                    if (issued >= S) {       // the slot's previous tile: free once the products that read it are done
                        ok = mbar_wait(&empty[slot], (uint32_t)((issued - S) / S) & 1u, abort_flag);
                        if (!ok) break;
                    }
                    mbar_arrive_expect_tx(&full[slot], TILE_BYTES);
                    tma_load_3d(tile0_ptr + (size_t)slot * TILE_BYTES, &tmV, &full[slot], 0, cur.row_base + ti * LG_TILE, 0);
                }
            }
        }
    } else if (warp == LGTC_MMA_WARP) {
        // =============================== tensor-core warp ===============================
        // (all lanes follow the same control flow; lane 0 issues the products)
        int it = 0, kk = 0;                 // tiles handed to the tensor core, non-empty items begun
        bool ok = true;
        for (uint32_t i = blockIdx.x; i < (uint32_t)p.items && ok; i += gridDim.x) {
            const LgItem cur = lg_item(p, s_nsel, i);
            if (cur.nt == 0) continue;
            const int ntiles = (cur.nt + LG_TILE - 1) / LG_TILE, j = kk & 1;
            ok = warp_wait(&p_ready[j], (uint32_t)(kk >> 1) & 1u, abort_flag);     // P[j] is written ...
            if (ok && kk >= 2) ok = warp_wait(&acc_free[j], (uint32_t)((kk - 2) >> 1) & 1u, abort_flag);   // ... item kk - 2's accumulator read out
            if (!ok) break;
            for (int ti = 0; ti < ntiles; ++ti, ++it) {
                const int s = it % S;
                ok = warp_wait(&full[s], (uint32_t)(it / S) & 1u, abort_flag);
                if (!ok) break;
                const uint32_t vbase = tile0 + s * TILE_BYTES;
                if ((ti + 1) * LG_TILE > cur.nt) {
                    // rows past the chunk's last slot hold whatever lies behind it (other slots, NaN patterns): clear them
                    // (whole 128-byte rows, so the swizzle does not matter), and let the tensor core see the zeros
                    const int first_bad = cur.nt - ti * LG_TILE;
                    for (int u = lane + first_bad * (HALVES * 8); u < LG_TILE * HALVES * 8; u += 32) {
                        const int r = u / (HALVES * 8), q = u % (HALVES * 8);
                        sts128_zero(vbase + (q >> 3) * HALF_BYTES + r * 128u + ((q & 7) << 4));
                    }
                    fence_proxy_async();
                }
                __syncwarp();
                if (lane == 0) {
                    tc_fence_after_sync();
                    const uint32_t acc = tmem + j * ACC_COLS;
                    // B: 16 rows (8 hi, 8 lo: 256 bytes apart) x 16 tokens (two 128-byte core matrices), 512 bytes per step;
                    // A: D components x 16 tokens: token rows of 128 bytes per 64-component half (halves HALF_BYTES
                    // apart), 8-row swizzle atoms 1024 bytes apart, 2048 bytes per step.  (The start address is the
                    // descriptor's low field, in 16-byte units: a step adds a constant.)
                    uint64_t bd = tc_smem_desc(p0 + j * pbytes + (uint32_t)(ti * STEPS) * 512u, 128u, 256u, 0u);
                    uint64_t ad = tc_smem_desc(vbase, (uint32_t)HALF_BYTES, 1024u, 2u);
#pragma unroll
                    for (int k4 = 0; k4 < STEPS; ++k4) {
                        tc_mma_f16(acc, ad, bd, IDESC, (ti | k4) != 0 ? 1u : 0u);
                        ad += (16 * 128) >> 4;
                        bd += 512 >> 4;
                    }
                    tc_commit(&empty[s]);                              // the slot is free when these products are done
                    if (ti == ntiles - 1) tc_commit(&done[j]);         // ... and so is the item
                }
                __syncwarp();
            }
            ++kk;
        }
    } else {
        // =============================== head warps: logits in, partials out ===============================
        // Per non-empty item k, in this order: wait for item k - 2's products (they read the P buffer and fill the
        // accumulator that item k takes over); turn item k's logits - requested one item earlier, so they are in
        // registers by now - into m, l and P[k & 1] and tell the driver; request item k + 1's logits; read item k - 2's
        // accumulator out and tell the driver that it is free.
        uint32_t cur_i = blockIdx.x;
        auto next_item = [&](LgItem& out) -> bool {           // the CTA's next non-empty item; empty ones are written on the way
            while (cur_i < (uint32_t)p.items) {
                const LgItem t = lg_item(p, s_nsel, cur_i);
                cur_i += gridDim.x;
                if (t.nt > 0) { out = t; return true; }
                const int nh = min(8, p.G - t.hb * 8);
                if (warp < nh) {
                    const size_t slot = ((size_t)t.b * p.Hq + t.g * p.G + t.hb * 8 + warp) * p.NC + t.c;
                    if (lane < D / 4) reinterpret_cast<float4*>(p.o_part + slot * D)[lane] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (lane == 0) { p.m_part[slot] = NEG_INF; p.l_part[slot] = 0.f; }
                }
            }
            return false;
        };
        // a lane owns token pairs (2u, 2u + 1), u = lane + 32 i: coalesced 8-byte loads
        auto pair_at = [&](const LgItem& im, int u) -> float2 {
            const int nh = min(8, p.G - im.hb * 8);
            float2 v = make_float2(NEG_INF, NEG_INF);
            if (warp < nh && 2 * u < im.nt) {
                const float* row = p.logits + ((size_t)im.b * p.Hq + im.g * p.G + im.hb * 8 + warp) * p.K + (size_t)im.c * p.chunk;
                if ((reinterpret_cast<uintptr_t>(row) & 7u) == 0 && 2 * u + 1 < im.nt) v = *reinterpret_cast<const float2*>(row + 2 * u);
                else { v.x = row[2 * u]; if (2 * u + 1 < im.nt) v.y = row[2 * u + 1]; }
            }
            return v;
        };
        // read-out of item k's accumulator by warps 0-3 (they hold the 128 lanes between them)
        auto read_out = [&](const LgItem& im, int k) {
            if (warp < 4) {
                const int j = k & 1;
                tc_fence_after_sync();
                // lane l of the tensor memory holds component l of the row (D = 128), or, for M = 64 products, lane
                // 32 w + i holds component 16 w + i (i < 16; lanes 16-31 of each quarter unused)
                uint32_t r[16];
                tmem_ld_32x16(tmem + ((uint32_t)(warp * 32) << 16) + j * ACC_COLS, r);
                tmem_ld_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_free[j]);
                const int h0 = im.g * p.G + im.hb * 8, nh = min(8, p.G - im.hb * 8);
                const int d = D == 128 ? warp * 32 + lane : warp * 16 + lane;
                if (D == 128 || lane < 16) {
                    const uint64_t keep = l2_evict_last_policy();      // the merge reads these lines next
#pragma unroll
                    for (int hh = 0; hh < 8; ++hh)
                        if (hh < nh)
                            st_global_hint(p.o_part + (((size_t)im.b * p.Hq + h0 + hh) * p.NC + im.c) * D + d,
                                           __uint_as_float(r[hh]) + __uint_as_float(r[8 + hh]), keep);
                }
            }
        };
        int k = 0;
        bool ok = true;
        LgItem itA, itN, q0, q1;                   // being built, next, and the two whose accumulators are still to be read (k - 2, k - 1)
        bool hasA = next_item(itA), hasN = false;
        float2 pre[4];
        if (hasA) {
#pragma unroll
            for (int q = 0; q < 4; ++q) pre[q] = pair_at(itA, lane + 32 * q);
        }
        while (hasA) {
            if (k >= 2) {
                ok = warp_wait(&done[k & 1], (uint32_t)((k - 2) >> 1) & 1u, abort_flag);
                if (!ok) break;
            }
            hasN = next_item(itN);
            const int j = k & 1, nt = itA.nt;
            const int nsteps = (nt + LG_TILE - 1) / LG_TILE * STEPS;
            const int h0 = itA.g * p.G + itA.hb * 8, nh = min(8, p.G - itA.hb * 8);
            const bool live = warp < nh;
            {
                // the chunk's first 256 slots are in registers already; the rest (chunks of more than 256 slots) is read
                // here, twice: once for the maximum, once for the weights
                float2 first[4];
                float mx = NEG_INF;
#pragma unroll
                for (int q = 0; q < 4; ++q) { first[q] = pre[q]; mx = fmaxf(mx, fmaxf(first[q].x, first[q].y)); }
                for (int u0 = 128; 2 * u0 < nt; u0 += 128) {
                    float2 v[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) v[q] = pair_at(itA, u0 + lane + 32 * q);
#pragma unroll
                    for (int q = 0; q < 4; ++q) mx = fmaxf(mx, fmaxf(v[q].x, v[q].y));
                }
#pragma unroll
                for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float msafe = (mx == NEG_INF) ? 0.f : mx;
                float sum = 0.f;
                uint8_t* const pj = p0_ptr + (size_t)j * pbytes;
                for (int u0 = 0; 2 * u0 < nsteps * 16; u0 += 128) {    // pair index u: step u / 8, position u % 8 in it
                    float2 sv[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) sv[q] = u0 == 0 ? first[q] : pair_at(itA, u0 + lane + 32 * q);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int u = u0 + lane + 32 * q;
                        if (2 * u >= nsteps * 16) break;
                        const float w0 = live ? fast_exp2((sv[q].x - msafe) * LOG2E) : 0.f;   // e^{-inf} = 0 for unused slots
                        const float w1 = live ? fast_exp2((sv[q].y - msafe) * LOG2E) : 0.f;
                        sum += w0 + w1;
                        const uint32_t hi = pack2<BF16>(w0, w1);
                        const float2 f = unpack2<BF16>(hi);
                        const uint32_t lo = pack2<BF16>(w0 - f.x, w1 - f.y);
                        // B operand of step kt, K-major without swizzle: rows 0-7 the heads' hi terms, rows 8-15 (256 bytes
                        // on) their lo terms; per row group two 128-byte core matrices (tokens 0-7, 8-15 of the step) of
                        // 8 rows x 16 bytes; this lane's pair is tokens 2 w8, 2 w8 + 1 of head `warp`
                        const int kt = u >> 3, w8 = u & 7;
                        uint8_t* dst = pj + (size_t)kt * 512 + (w8 >> 2) * 128 + warp * 16 + (w8 & 3) * 4;
                        *reinterpret_cast<uint32_t*>(dst) = hi;
                        *reinterpret_cast<uint32_t*>(dst + 256) = lo;
                    }
                }
#pragma unroll
                for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                if (lane == 0 && live) {
                    const size_t slot = ((size_t)itA.b * p.Hq + h0 + warp) * p.NC + itA.c;
                    p.m_part[slot] = mx;
                    p.l_part[slot] = sum;
                }
            }
            fence_proxy_async();              // the tensor core reads P through the asynchronous proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_ready[j]);
            if (hasN) {
#pragma unroll
                for (int q = 0; q < 4; ++q) pre[q] = pair_at(itN, lane + 32 * q);
            }
            if (k >= 2) read_out(q0, k - 2);
            q0 = q1; q1 = itA;
            itA = itN; hasA = hasN;
            ++k;
        }
        // the last two items' accumulators
        for (int kk = max(k - 2, 0); kk < k && ok; ++kk) {
            ok = warp_wait(&done[kk & 1], (uint32_t)(kk >> 1) & 1u, abort_flag);
            if (ok) read_out(kk == k - 1 ? q1 : q0, kk);
        }
    }
    __syncthreads();
    if (tid == LGTC_LOAD_WARP * 32 && *abort_flag) {
        // unwinding: copies into this CTA's shared memory may still be on their way
        for (int i = max(0, issued - S); i < issued; ++i) {
            int dummy = 0;
            mbar_wait(&full[i % S], (uint32_t)(i / S) & 1u, &dummy);
        }
        if (p.status) atomicOr(p.status, HG_DEV_WAIT_TIMEOUT);
    }
    __syncthreads();
    if (warp == LGTC_MMA_WARP) tmem_dealloc(tmem, LGTC_TMEM_COLS);
}

}  // namespace hg
