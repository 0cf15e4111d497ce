// Split-KV decode attention partials over a paged 16-bit KV pool (sm_100a).
//
// One CTA per work item (sequence b, KV head g [, block of 8 query heads], chunk c).  A producer
// warp streams the item's K and V tiles (64 tokens x D, 128-byte-swizzled) from HBM into a ring of
// shared-memory stages with TMA tensor loads; four consumer warps each own 16 token rows of every
// tile and keep a private online-softmax state (running max, exp-sum, un-normalised output), which
// is merged across warps once at the end.  K_j and V_j alternate in the ring, so the logits never
// leave the chip.
//
//   MODE_MHA    one query head per KV head: dot products on CUDA cores, fp32 throughout.
//   MODE_GQA    up to 8 query heads share the KV head: S^T = K q^T and O^T = V^T P^T on warp-level
//               tensor-core MMAs (tokens are the M dimension, heads the N dimension, nothing padded
//               for a group of 8).  P is fed as hi + lo 16-bit terms, so its rounding error is ~2^-17
//               (bf16) / ~2^-22 (fp16) instead of one 16-bit ulp.
//   MODE_PROBE  same loads, no attention math: folds the slice's bytes into a checksum.
#pragma once

#include "hg_device.cuh"

namespace hg {

constexpr int TILE_T = 64;             // tokens per tile
constexpr int CONSUMER_WARPS = 4;
constexpr int CONSUMER_THREADS = CONSUMER_WARPS * 32;
constexpr int THREADS = CONSUMER_THREADS + 32;
constexpr int MAX_STAGES = 12;
constexpr int MAX_CHUNK_PAGES = 1024;
constexpr int HALF_BYTES = TILE_T * 128;  // one 64-element (128-byte) column half of a tile

enum { MODE_MHA = 0, MODE_GQA = 1, MODE_PROBE = 2 };

struct PartialParams {
    const void* q;
    const int32_t* seq_lens;
    const int32_t* tok_begin;
    const int32_t* tok_end;
    const int32_t* block_table;
    float* o_part;
    float* m_part;
    float* l_part;
    uint32_t* sink;
    int32_t* status;
    int B, Hq, Hkv, G;
    int page_size, page_shift, max_pages, num_pages;
    int C, NC, stages, head_blocks;
    int perm0, perm1, perm2;  // tensor-map dim 1+i carries logical coordinate perm_i: 0 = token-in-page, 1 = head, 2 = page
    float scale_log2;         // logit scale * log2(e)
};

struct Control {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    int abort_flag;
    uint32_t probe_acc;
    int pages[MAX_CHUNK_PAGES];
    float red_m[32];
    float red_l[32];
};

__device__ __forceinline__ int pick3(int k, int a, int b, int c) { return k == 0 ? a : (k == 1 ? b : c); }

// All lanes wait; the verdict is made warp-uniform so that no lane leaves a loop alone.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const bool ok = mbar_wait(bar, parity, abort_flag);
    return __all_sync(0xffffffffu, ok);
}

template <int D, bool BF16, int MODE>
__global__ void __launch_bounds__(THREADS) partial_kernel(const __grid_constant__ CUtensorMap tmK,
                                                          const __grid_constant__ CUtensorMap tmV,
                                                          const PartialParams p) {
    constexpr int HALVES = D / 64;
    constexpr int STAGE_BYTES = HALVES * HALF_BYTES;
    constexpr int NV = 8 * HALVES;     // MHA: d-components owned by a lane
    constexpr int KSTEPS = D / 16;     // GQA: 16-wide steps along d
    const float NEG_INF = __int_as_float(0xff800000);

    extern __shared__ uint8_t smem_raw[];
    __shared__ Control ctl;
    const uint32_t stage0 = (smem_u32(smem_raw) + 1023u) & ~1023u;   // the swizzle pattern is anchored at 1024 bytes
    uint8_t* const stage0_ptr = smem_raw + (stage0 - smem_u32(smem_raw));

#if __CUDA_ARCH__ >= 900
    cudaTriggerProgrammaticLaunchCompletion();   // a dependent merge launch may be scheduled while this grid drains
#endif
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c = blockIdx.x;
    const int g = blockIdx.y / p.head_blocks, hb = blockIdx.y % p.head_blocks;
    const int b = blockIdx.z;

    // ---- the item's token range --------------------------------------------------------------
    const int L = p.seq_lens[b];
    const int tb = max(p.tok_begin[b], 0);
    const int te = min(p.tok_end[b], L);
    const int first = tb / p.C;
    const int lo = max((first + c) * p.C, tb);
    const int hi = min((first + c + 1) * p.C, te);

    const int nheads = (MODE == MODE_GQA) ? min(8, p.G - hb * 8) : 1;
    const int h0 = (MODE == MODE_GQA) ? g * p.G + hb * 8 : g;   // first query head of this item

    if (te <= tb || lo >= hi) {            // empty chunk slot: neutral element
        if constexpr (MODE == MODE_PROBE) {
            if (tid == 0) p.sink[((size_t)b * p.Hkv + g) * p.NC + c] = 0u;
        } else {
            for (int i = tid; i < nheads * D; i += THREADS)
                p.o_part[(((size_t)b * p.Hq + h0 + i / D) * p.NC + c) * D + i % D] = 0.f;
            if (tid < nheads) {
                p.m_part[((size_t)b * p.Hq + h0 + tid) * p.NC + c] = NEG_INF;
                p.l_part[((size_t)b * p.Hq + h0 + tid) * p.NC + c] = 0.f;
            }
        }
        return;
    }

    // a wait already timed out in this call (or the caller left the word set): do not queue behind it
    if (p.status && *reinterpret_cast<volatile int32_t*>(p.status) == HG_DEV_WAIT_TIMEOUT) {
        if constexpr (MODE != MODE_PROBE) {
            if (tid < nheads) p.m_part[((size_t)b * p.Hq + h0 + tid) * p.NC + c] = __int_as_float(0x7fc00000);
        }
        return;
    }

    const int tile0 = lo / TILE_T;
    const int ntiles = (hi + TILE_T - 1) / TILE_T - tile0;
    const int page0 = (tile0 * TILE_T) >> p.page_shift;
    const int npages = (((tile0 + ntiles) * TILE_T - 1) >> p.page_shift) + 1 - page0;
    const int n_iter = 2 * ntiles;   // K_0, V_0, K_1, V_1, ...

    // ---- set-up: barriers and the physical page ids of this chunk -------------------------------
    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&ctl.full[s], 1);
            mbar_init(&ctl.empty[s], CONSUMER_WARPS);
        }
        ctl.abort_flag = 0;
        ctl.probe_acc = 0u;
        fence_barrier_init();
    }
    for (int i = tid; i < npages && i < MAX_CHUNK_PAGES; i += THREADS) {
        const int pg = page0 + i;
        int phys = -1;
        if (pg * p.page_size < hi && (pg + 1) * p.page_size > lo) {
            if (pg < p.max_pages)
                phys = p.block_table ? p.block_table[(size_t)b * p.max_pages + pg] : b * p.max_pages + pg;
            if (phys < 0 || phys >= p.num_pages) {
                if (p.status) atomicMax(p.status, HG_DEV_BAD_PAGE);
                phys = -1;
            }
        }
        ctl.pages[i] = phys;
    }
    __syncthreads();

    volatile int* abort_flag = &ctl.abort_flag;

    // consumer state (only the active mode's survives compilation); parked in shared memory after the loop
    float mha_m = NEG_INF, mha_l = 0.f, mha_o[NV];
    float gqa_m[2] = {NEG_INF, NEG_INF}, gqa_l[2] = {0.f, 0.f}, gqa_o[KSTEPS][4];
    uint32_t probe_x = 0u;
#pragma unroll
    for (int i = 0; i < NV; ++i) mha_o[i] = 0.f;
#pragma unroll
    for (int i = 0; i < KSTEPS; ++i) { gqa_o[i][0] = gqa_o[i][1] = gqa_o[i][2] = gqa_o[i][3] = 0.f; }

    const int row0 = warp * 16;                  // a consumer warp's rows within every tile
    const int gi = lane >> 3, li = lane & 7;     // MHA: 8 lanes share a token row; 4 row groups per warp
    const int quad = lane >> 2, tq = lane & 3;   // GQA: MMA fragment coordinates

    if (warp == CONSUMER_WARPS) {
        // ======================= producer warp =======================
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
        const uint64_t policy = l2_evict_first_policy();
        const int rows = p.page_size >= TILE_T ? TILE_T : p.page_size;
        const int nbox = p.page_size >= TILE_T ? 1 : (TILE_T >> p.page_shift);
        const int j = lane / HALVES, h = lane % HALVES;
        int issued = 0;
        for (int it = 0; it < n_iter; ++it) {
            const int s = it % p.stages;
            const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
            int okw = 1;
            if (lane == 0) okw = mbar_wait(&ctl.empty[s], ph ^ 1u, abort_flag) ? 1 : 0;
            okw = __shfl_sync(0xffffffffu, okw, 0);
            if (!okw) break;
            const int tokbase = (tile0 + (it >> 1)) * TILE_T;
            const int t0j = tokbase + j * rows;
            int phys = -1;
            if (j < nbox && t0j < hi && t0j + rows > lo) phys = ctl.pages[(t0j >> p.page_shift) - page0];
            const uint32_t nvalid = __popc(__ballot_sync(0xffffffffu, phys >= 0 && h == 0));
            if (lane == 0) mbar_arrive_expect_tx(&ctl.full[s], nvalid * (uint32_t)rows * 128u * HALVES);
            __syncwarp();
            if (phys >= 0) {
                const int tin = t0j & (p.page_size - 1);
                uint8_t* dst = stage0_ptr + (size_t)s * STAGE_BYTES + h * HALF_BYTES + j * rows * 128;
                tma_load_4d(dst, (it & 1) ? &tmV : &tmK, &ctl.full[s], h * 64, pick3(p.perm0, tin, g, phys),
                            pick3(p.perm1, tin, g, phys), pick3(p.perm2, tin, g, phys), policy);
            }
            issued = it + 1;
        }
        if (*abort_flag && lane == 0) {
            // unwinding: do not leave the CTA while copies into its shared memory may still land
            for (int it = max(0, issued - p.stages); it < issued; ++it) {
                int dummy = 0;
                mbar_wait(&ctl.full[it % p.stages], (uint32_t)(it / p.stages) & 1u, &dummy);
            }
        }
    } else if constexpr (MODE == MODE_PROBE) {
        // ======================= probe consumers =======================
        for (int it = 0; it < n_iter; ++it) {
            const int s = it % p.stages;
            if (!warp_wait(&ctl.full[s], (uint32_t)(it / p.stages) & 1u, abort_flag)) break;
            const uint32_t base = stage0 + s * STAGE_BYTES;
            const int tokbase = (tile0 + (it >> 1)) * TILE_T;
#pragma unroll
            for (int i = 0; i < 4 * HALVES; ++i) {
                // 16 rows x HALVES x 8 chunks per warp; a quarter-warp reads one 128-byte row segment
                const int idx = i * 32 + lane;
                const int r = row0 + (idx >> 3) % 16, hh = (idx >> 3) / 16;
                const int t = tokbase + r;
                if (t >= lo && t < hi) {
                    uint4 v = lds128(base + hh * HALF_BYTES + r * 128 + ((idx & 7) << 4));
                    probe_x ^= v.x ^ v.y ^ v.z ^ v.w;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl.empty[s]);
        }
    } else if constexpr (MODE == MODE_MHA) {
        // ======================= MHA consumers (CUDA cores) =======================
        float qf[NV];
        {
            const uint16_t* qrow = reinterpret_cast<const uint16_t*>(p.q) + ((size_t)b * p.Hq + h0) * D;
#pragma unroll
            for (int hh = 0; hh < HALVES; ++hh) {
                uint4 raw = *reinterpret_cast<const uint4*>(qrow + hh * 64 + li * 8);
                float2 a = unpack2<BF16>(raw.x), bb = unpack2<BF16>(raw.y), cc = unpack2<BF16>(raw.z),
                       dd = unpack2<BF16>(raw.w);
                qf[hh * 8 + 0] = a.x; qf[hh * 8 + 1] = a.y; qf[hh * 8 + 2] = bb.x; qf[hh * 8 + 3] = bb.y;
                qf[hh * 8 + 4] = cc.x; qf[hh * 8 + 5] = cc.y; qf[hh * 8 + 6] = dd.x; qf[hh * 8 + 7] = dd.y;
            }
        }
        const int rbase = row0 + gi * 4;      // this lane group's 4 rows
        for (int jt = 0; jt < ntiles; ++jt) {
            const int tokbase = (tile0 + jt) * TILE_T;
            bool valid[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) { const int t = tokbase + rbase + k; valid[k] = t >= lo && t < hi; }

            // ---- K tile: 4 logits per lane group ----
            int it = 2 * jt, s = it % p.stages;
            if (!warp_wait(&ctl.full[s], (uint32_t)(it / p.stages) & 1u, abort_flag)) break;
            uint32_t base = stage0 + s * STAGE_BYTES;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int r = rbase + k;
#pragma unroll
                for (int hh = 0; hh < HALVES; ++hh) {
                    uint4 raw = lds128(base + hh * HALF_BYTES + r * 128 + ((li ^ (r & 7)) << 4));
                    float2 a = unpack2<BF16>(raw.x), bb = unpack2<BF16>(raw.y), cc = unpack2<BF16>(raw.z),
                           dd = unpack2<BF16>(raw.w);
                    const float* qq = &qf[hh * 8];
                    acc[k] = fmaf(a.x, qq[0], acc[k]); acc[k] = fmaf(a.y, qq[1], acc[k]);
                    acc[k] = fmaf(bb.x, qq[2], acc[k]); acc[k] = fmaf(bb.y, qq[3], acc[k]);
                    acc[k] = fmaf(cc.x, qq[4], acc[k]); acc[k] = fmaf(cc.y, qq[5], acc[k]);
                    acc[k] = fmaf(dd.x, qq[6], acc[k]); acc[k] = fmaf(dd.y, qq[7], acc[k]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl.empty[s]);
            float s2[4], mx = NEG_INF;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float v = acc[k];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                s2[k] = valid[k] ? v * p.scale_log2 : NEG_INF;
                mx = fmaxf(mx, s2[k]);
            }
            const float m_new = fmaxf(mha_m, mx);
            const float m_safe = (m_new == NEG_INF) ? 0.f : m_new;
            const float corr = fast_exp2(mha_m - m_safe);
            float pk[4], psum = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) { pk[k] = fast_exp2(s2[k] - m_safe); psum += pk[k]; }
            mha_l = mha_l * corr + psum;
            mha_m = m_new;

            // ---- V tile: o = o * corr + sum_k p_k V_k ----
            it = 2 * jt + 1; s = it % p.stages;
            if (!warp_wait(&ctl.full[s], (uint32_t)(it / p.stages) & 1u, abort_flag)) break;
            base = stage0 + s * STAGE_BYTES;
#pragma unroll
            for (int i = 0; i < NV; ++i) mha_o[i] *= corr;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int r = rbase + k;
#pragma unroll
                for (int hh = 0; hh < HALVES; ++hh) {
                    uint4 raw = make_uint4(0u, 0u, 0u, 0u);      // rows outside the slice never enter the sum
                    if (valid[k]) raw = lds128(base + hh * HALF_BYTES + r * 128 + ((li ^ (r & 7)) << 4));
                    float2 a = unpack2<BF16>(raw.x), bb = unpack2<BF16>(raw.y), cc = unpack2<BF16>(raw.z),
                           dd = unpack2<BF16>(raw.w);
                    float* oo = &mha_o[hh * 8];
                    oo[0] = fmaf(pk[k], a.x, oo[0]); oo[1] = fmaf(pk[k], a.y, oo[1]);
                    oo[2] = fmaf(pk[k], bb.x, oo[2]); oo[3] = fmaf(pk[k], bb.y, oo[3]);
                    oo[4] = fmaf(pk[k], cc.x, oo[4]); oo[5] = fmaf(pk[k], cc.y, oo[5]);
                    oo[6] = fmaf(pk[k], dd.x, oo[6]); oo[7] = fmaf(pk[k], dd.y, oo[7]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl.empty[s]);
        }
    } else {
        // ======================= GQA consumers (tensor cores) =======================
        // q^T as the B operand of S^T = K q^T: b0 = q[head quad][16 ks + 2 tq + {0,1}], b1 = the same + 8
        uint32_t qb[KSTEPS][2];
        {
            const bool live = hb * 8 + quad < p.G;
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
                reinterpret_cast<const uint16_t*>(p.q) + ((size_t)b * p.Hq + (live ? h0 + quad : h0)) * D);
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                qb[ks][0] = live ? qrow[ks * 8 + tq] : 0u;
                qb[ks][1] = live ? qrow[ks * 8 + 4 + tq] : 0u;
            }
        }
        // ldmatrix row addresses (within a tile) for this lane
        const int a_row = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;   // K: matrices (rows, rows+8) x (k lo, k hi)
        const int a_kc = lane >> 4;
        const int v_row = row0 + (lane & 7) + (lane >> 4) * 8;         // V^T: matrices (d lo, d hi) x (tok, tok+8)
        const int v_dc = (lane >> 3) & 1;

        for (int jt = 0; jt < ntiles; ++jt) {
            const int tokbase = (tile0 + jt) * TILE_T;
            const int tA = tokbase + row0 + quad, tB = tA + 8;
            const bool vA = tA >= lo && tA < hi, vB = tB >= lo && tB < hi;
            const bool edge = tokbase < lo || tokbase + TILE_T > hi;

            // ---- S^T (16 tokens x 8 heads) ----
            int it = 2 * jt, s = it % p.stages;
            if (!warp_wait(&ctl.full[s], (uint32_t)(it / p.stages) & 1u, abort_flag)) break;
            uint32_t base = stage0 + s * STAGE_BYTES;
            float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                const int ch = 2 * ks + a_kc;   // 16-byte chunk index along d
                uint32_t a[4];
                ldmatrix_x4(a, base + (ch >> 3) * HALF_BYTES + a_row * 128 + (((ch & 7) ^ (a_row & 7)) << 4));
                mma_16816<BF16>(sc, a, qb[ks][0], qb[ks][1]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl.empty[s]);

            // sc[0], sc[1]: token tA, heads 2tq, 2tq+1; sc[2], sc[3]: token tB
            float s2[4];
            s2[0] = vA ? sc[0] * p.scale_log2 : NEG_INF; s2[1] = vA ? sc[1] * p.scale_log2 : NEG_INF;
            s2[2] = vB ? sc[2] * p.scale_log2 : NEG_INF; s2[3] = vB ? sc[3] * p.scale_log2 : NEG_INF;
            float mx[2] = {fmaxf(s2[0], s2[2]), fmaxf(s2[1], s2[3])};
#pragma unroll
            for (int o = 4; o <= 16; o <<= 1) {
                mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], o));
                mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], o));
            }
            float corr[2], msafe[2];
#pragma unroll
            for (int hc = 0; hc < 2; ++hc) {
                const float m_new = fmaxf(gqa_m[hc], mx[hc]);
                msafe[hc] = (m_new == NEG_INF) ? 0.f : m_new;
                corr[hc] = fast_exp2(gqa_m[hc] - msafe[hc]);
                gqa_m[hc] = m_new;
            }
            float pr[4];
            pr[0] = fast_exp2(s2[0] - msafe[0]); pr[1] = fast_exp2(s2[1] - msafe[1]);
            pr[2] = fast_exp2(s2[2] - msafe[0]); pr[3] = fast_exp2(s2[3] - msafe[1]);
            gqa_l[0] = gqa_l[0] * corr[0] + pr[0] + pr[2];   // per-lane sums over its own two token rows
            gqa_l[1] = gqa_l[1] * corr[1] + pr[1] + pr[3];

            // P^T as the B operand of O^T += V^T P^T, as hi + lo 16-bit terms
            const uint32_t hiA = pack2<BF16>(pr[0], pr[1]), hiB = pack2<BF16>(pr[2], pr[3]);
            const float2 fA = unpack2<BF16>(hiA), fB = unpack2<BF16>(hiB);
            const uint32_t loA = pack2<BF16>(pr[0] - fA.x, pr[1] - fA.y), loB = pack2<BF16>(pr[2] - fB.x, pr[3] - fB.y);
            const uint32_t bh0 = movmatrix_trans(hiA), bh1 = movmatrix_trans(hiB);
            const uint32_t bl0 = movmatrix_trans(loA), bl1 = movmatrix_trans(loB);

            // ---- O^T ----
            it = 2 * jt + 1; s = it % p.stages;
            if (!warp_wait(&ctl.full[s], (uint32_t)(it / p.stages) & 1u, abort_flag)) break;
            base = stage0 + s * STAGE_BYTES;
            if (edge) {
                // rows outside the slice may hold anything (even NaN patterns): clear this warp's copies
                for (int i = lane; i < 16 * 8 * HALVES; i += 32) {
                    const int r = row0 + (i / (8 * HALVES)), ch = i % (8 * HALVES);
                    const int t = tokbase + r;
                    if (t < lo || t >= hi) sts128_zero(base + (ch >> 3) * HALF_BYTES + r * 128 + ((ch & 7) << 4));
                }
                __syncwarp();
            }
#pragma unroll
            for (int mt = 0; mt < KSTEPS; ++mt) {
                gqa_o[mt][0] *= corr[0]; gqa_o[mt][1] *= corr[1]; gqa_o[mt][2] *= corr[0]; gqa_o[mt][3] *= corr[1];
                const int ch = 2 * mt + v_dc;
                uint32_t a[4];
                ldmatrix_x4_trans(a, base + (ch >> 3) * HALF_BYTES + v_row * 128 + (((ch & 7) ^ (v_row & 7)) << 4));
                mma_16816<BF16>(gqa_o[mt], a, bh0, bh1);
                mma_16816<BF16>(gqa_o[mt], a, bl0, bl1);
            }
            if (edge) fence_proxy_async();   // the generic-proxy stores above precede the next TMA write to this stage
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl.empty[s]);
        }
#pragma unroll
        for (int o = 4; o <= 16; o <<= 1) {
            gqa_l[0] += __shfl_xor_sync(0xffffffffu, gqa_l[0], o);
            gqa_l[1] += __shfl_xor_sync(0xffffffffu, gqa_l[1], o);
        }
    }

    // ---- every issued tile has landed and been read: the stage memory becomes the reduction buffer ----
    __syncthreads();
    float* const red_o = reinterpret_cast<float*>(stage0_ptr);
    if (warp < CONSUMER_WARPS && !*abort_flag) {
        if constexpr (MODE == MODE_PROBE) {
#pragma unroll
            for (int o = 16; o; o >>= 1) probe_x ^= __shfl_xor_sync(0xffffffffu, probe_x, o);
            if (lane == 0) atomicXor(&ctl.probe_acc, probe_x);
        } else if constexpr (MODE == MODE_MHA) {
            const int slot = warp * 4 + gi;                       // red_o [16 row groups][D]
            if (li == 0) { ctl.red_m[slot] = mha_m; ctl.red_l[slot] = mha_l; }
#pragma unroll
            for (int hh = 0; hh < HALVES; ++hh) {
                float4* dst = reinterpret_cast<float4*>(red_o + slot * D + hh * 64 + li * 8);
                dst[0] = make_float4(mha_o[hh * 8 + 0], mha_o[hh * 8 + 1], mha_o[hh * 8 + 2], mha_o[hh * 8 + 3]);
                dst[1] = make_float4(mha_o[hh * 8 + 4], mha_o[hh * 8 + 5], mha_o[hh * 8 + 6], mha_o[hh * 8 + 7]);
            }
        } else {
            if (quad == 0) {                                      // red_o [4 warps][8 heads][D]
                ctl.red_m[warp * 8 + 2 * tq] = gqa_m[0]; ctl.red_m[warp * 8 + 2 * tq + 1] = gqa_m[1];
                ctl.red_l[warp * 8 + 2 * tq] = gqa_l[0]; ctl.red_l[warp * 8 + 2 * tq + 1] = gqa_l[1];
            }
            float* w = red_o + (size_t)warp * 8 * D;
#pragma unroll
            for (int mt = 0; mt < KSTEPS; ++mt) {
                const int d0 = mt * 16 + quad;
                w[(2 * tq) * D + d0] = gqa_o[mt][0];
                w[(2 * tq + 1) * D + d0] = gqa_o[mt][1];
                w[(2 * tq) * D + d0 + 8] = gqa_o[mt][2];
                w[(2 * tq + 1) * D + d0 + 8] = gqa_o[mt][3];
            }
        }
    }
    __syncthreads();

    if (*abort_flag) {
        if (p.status && tid == 0) atomicMax(p.status, HG_DEV_WAIT_TIMEOUT);
        if constexpr (MODE != MODE_PROBE) {
            if (tid < nheads) p.m_part[((size_t)b * p.Hq + h0 + tid) * p.NC + c] = __int_as_float(0x7fc00000);
        }
        return;
    }

    if constexpr (MODE == MODE_PROBE) {
        if (tid == 0) p.sink[((size_t)b * p.Hkv + g) * p.NC + c] = ctl.probe_acc;
    } else {
        constexpr int NSRC = (MODE == MODE_MHA) ? 16 : CONSUMER_WARPS;       // states to merge per head
        constexpr int HSTRIDE = (MODE == MODE_MHA) ? 0 : D;                  // red_o: [src][head][D]
        constexpr int SSTRIDE = (MODE == MODE_MHA) ? D : 8 * D;
        constexpr float LN2 = 0.6931471805599453f;
        for (int i = tid; i < nheads * D; i += THREADS) {
            const int hh = i / D, d = i % D;
            float M = NEG_INF;
#pragma unroll
            for (int sidx = 0; sidx < NSRC; ++sidx) M = fmaxf(M, ctl.red_m[(MODE == MODE_MHA) ? sidx : sidx * 8 + hh]);
            float accv = 0.f, lsum = 0.f;
#pragma unroll
            for (int sidx = 0; sidx < NSRC; ++sidx) {
                const int mi = (MODE == MODE_MHA) ? sidx : sidx * 8 + hh;
                const float w = fast_exp2(ctl.red_m[mi] - M);      // -inf states weigh 0; M is finite here
                accv = fmaf(w, red_o[sidx * SSTRIDE + hh * HSTRIDE + d], accv);
                lsum = fmaf(w, ctl.red_l[mi], lsum);
            }
            const size_t slot = ((size_t)b * p.Hq + h0 + hh) * p.NC + c;
            p.o_part[slot * D + d] = accv;
            if (d == 0) { p.m_part[slot] = M * LN2; p.l_part[slot] = lsum; }
        }
    }
}

}  // namespace hg
