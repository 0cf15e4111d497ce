// Softmax partial from host-computed logits and gathered V rows (sm_100a): the device side of the
// paper's CPU -> GPU hand-off.  The host ships, per (sequence, query head), the scaled logits of its
// selected tokens and, per (sequence, KV head), the matching V rows; this kernel turns every chunk of
// them into the same (m, l, o) partial that hg_attn_partial produces for GPU-resident tokens, so the
// merge kernel treats both sides alike.  q.K^T is skipped; only V is streamed.
//
// Grid (chunk, KV head, sequence), 256 threads.  Thread 0 keeps a ring of V tiles (64 rows x D, one TMA
// tensor load each, 128-byte swizzled: the layout hg_attn_partial uses) in flight from the first
// instruction on.  Meanwhile, per block of up to 8 query heads of the group, warp h reads head h's logits of the
// chunk straight into registers, finds their maximum m, forms p = e^{s - m} and their sum l, and leaves p in
// shared memory already split into hi + lo 16-bit terms and ordered as the B fragments of
//     O^T [D x heads] += V^T [D x tokens] . P^T [tokens x heads]        (mma.sync m16n8k16, fp32 accumulate),
// the contraction of hg_attn_partial's group-query path, which every group size takes here (a single head
// wastes seven of the eight columns; the tensor pipe has the room, the path stays bound by the V stream).
// The 8 warps split D (16 components each at D = 128; at D = 64 two sets of four warps take alternate
// 16-token steps and add up at the end), so no V element is read from shared memory twice and nothing
// is reduced across warps.  Because m is known before the first product, nothing is ever rescaled.
// Groups of more than 8 heads stream the chunk's V tiles once per head block.
#pragma once

#include "hg_device.cuh"

namespace hg {

constexpr int LG_THREADS = 256;
constexpr int LG_WARPS = LG_THREADS / 32;
constexpr int LG_MAX_CHUNK = 1024;    // selected tokens per chunk
constexpr int LG_TILE = 64;           // V rows per tile
constexpr int LG_MIN_CTAS = 5;        // per SM
// Tiles in flight per CTA: two of 16 KB (D = 128) or three of 8 KB (D = 64, where two and four measured slower).  A CTA streams nothing while it turns its
// chunk's logits into fragments, so what keeps the V stream going is the number of CTAs that share an SM, not the
// depth of one CTA's ring: five CTAs with two tiles each run 10-14 % faster than three with three.
template <int D>
__host__ __device__ constexpr int lg_stages() { return D == 128 ? 2 : 3; }

struct LogitsParams {
    const float* logits;      // [B][Hq][K]
    const int32_t* n_sel;     // [B]
    float* o_part;            // [B][Hq][NC][D]
    float* m_part;            // [B][Hq][NC]
    float* l_part;
    int32_t* status;          // optional: HG_DEV_WAIT_TIMEOUT when a bounded wait ran out
    int B, Hq, Hkv, G, K, chunk, NC;
    // the tcgen05 kernel only: V tiles in its ring, blocks of 8 heads per group, work items in all
    int stages, head_blocks;
    long long items;
};

// Dynamic shared memory: [lg_stages<D>()] V tiles (64 x D x 2 bytes, 1024-byte aligned), then the P fragments
// (chunk / 16 steps x 32 lanes x 4 words), then, at D = 64, the second warp set's accumulators.
template <int D>
constexpr size_t logits_smem_bytes(int chunk) {
    return 1024 + (size_t)lg_stages<D>() * LG_TILE * D * 2 + (size_t)((chunk + LG_TILE - 1) / LG_TILE * LG_TILE / 16) * 512 +
           (D == 64 ? 4 * 32 * 4 * sizeof(float) : 0);
}

template <int D, bool BF16>
__global__ void __launch_bounds__(LG_THREADS, LG_MIN_CTAS) logits_partial_kernel(const __grid_constant__ CUtensorMap tmV, const LogitsParams p) {
    constexpr int TILE_BYTES = LG_TILE * D * 2;
    constexpr int LG_STAGES = lg_stages<D>();
    constexpr int MT = D / 16;                        // 16-component blocks of D: one per warp of a set
    constexpr int SETS = LG_WARPS / MT;               // warp sets taking alternate 16-token steps (1 or 2)
    constexpr float LOG2E = 1.4426950408889634f;
    const float NEG_INF = __int_as_float(0xff800000);

    extern __shared__ uint8_t lg_raw[];
    __shared__ uint64_t full[LG_STAGES], empty[LG_STAGES];
    __shared__ float s_m[8], s_l[8];
    __shared__ int abort_flag_s;
    const uint32_t tile0 = (smem_u32(lg_raw) + 1023u) & ~1023u;
    uint8_t* const tile0_ptr = lg_raw + (tile0 - smem_u32(lg_raw));
    uint4* const s_frag = reinterpret_cast<uint4*>(tile0_ptr + LG_STAGES * TILE_BYTES);       // [step][lane]

    const int c = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int quad = lane >> 2, tq = lane & 3;
    const int n = min(max(p.n_sel[b], 0), p.K);
    const int t0 = c * p.chunk, t1 = min(t0 + p.chunk, n);
    const int nt = max(t1 - t0, 0);                                   // slots of this chunk in use
    const int ntiles = (nt + LG_TILE - 1) / LG_TILE, nsteps = ntiles * (LG_TILE / 16);
    const int head_blocks = (p.G + 7) / 8;
    const int total = ntiles * head_blocks;                           // tiles this CTA streams, head block after head block
    const int row_base = (b * p.Hkv + g) * p.K + t0;                  // first V row of the chunk in the [B*Hkv*K][D] view
    volatile int* abort_flag = &abort_flag_s;

    if (tid == 0) {
        prefetch_tensormap(&tmV);
        for (int s = 0; s < LG_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], LG_WARPS); }
        abort_flag_s = 0;
        fence_barrier_init();
    }
    __syncthreads();
    auto issue = [&](int i) {                                          // tile i of the CTA's sequence into slot i % LG_STAGES
        const int s = i % LG_STAGES;
        mbar_arrive_expect_tx(&full[s], TILE_BYTES);
        tma_load_3d(tile0_ptr + (size_t)s * TILE_BYTES, &tmV, &full[s], 0, row_base + (i % ntiles) * LG_TILE, 0);
    };
    int issued = 0;                                                    // (thread 0) tiles requested so far
    if (tid == 0)
        for (; issued < total && issued < LG_STAGES; ++issued) issue(issued);

    // ldmatrix.trans addresses of this lane: matrices (d lo, d hi) x (tok, tok + 8) of its warp's 16 components
    const int mt = warp % MT, set = warp / MT;
    const int v_row = (lane & 7) + (lane >> 4) * 8, v_dc = (lane >> 3) & 1;
    const int ch = 2 * mt + v_dc;                                      // 16-byte chunk along d
    const uint32_t v_off = (uint32_t)(ch >> 3) * (128u * LG_TILE) + (uint32_t)v_row * 128u + (uint32_t)(((ch & 7) ^ (v_row & 7)) << 4);

    int it = 0;                                                        // tiles consumed so far
    for (int hb = 0; hb < head_blocks; ++hb) {
        const int h0 = g * p.G + hb * 8, nh = min(8, p.G - hb * 8);
        // ---- warp h: head h's logits -> m, l and the P fragments -------------------------------------------
        if (hb > 0) __syncthreads();          // the previous block's m and l have been written out (reached by all: see below)
        {
            // a lane owns token pairs (2u, 2u + 1), u = lane + 32 i: coalesced 8-byte loads, once for the maximum and
            // once more (out of the cache) for the weights; the first 256 slots - the whole chunk, at the usual chunk
            // size - are kept in registers instead
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
            float2 first[4];                                           // the chunk's first 256 slots stay in registers
#pragma unroll
            for (int j = 0; j < 4; ++j) first[j] = pair_at(lane + 32 * j);
#pragma unroll
            for (int j = 0; j < 4; ++j) mx = fmaxf(mx, fmaxf(first[j].x, first[j].y));
            for (int u0 = 128; 2 * u0 < nt; u0 += 128) {               // four independent loads in flight per lane
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
            uint32_t* const fw = reinterpret_cast<uint32_t*>(s_frag);
            for (int u0 = 0; 2 * u0 < nsteps * 16; u0 += 128) {        // pair index u: step u / 8, position u % 8 in it
                float2 sv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) sv[j] = u0 == 0 ? first[j] : pair_at(u0 + lane + 32 * j);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int u = u0 + lane + 32 * j;
                    if (2 * u >= nsteps * 16) break;
                    const float p0 = live ? fast_exp2((sv[j].x - msafe) * LOG2E) : 0.f;   // e^{-inf} = 0 for unused slots
                    const float p1 = live ? fast_exp2((sv[j].y - msafe) * LOG2E) : 0.f;
                    sum += p0 + p1;
                    const uint32_t hi = pack2<BF16>(p0, p1);
                    const float2 f = unpack2<BF16>(hi);
                    const uint32_t lo = pack2<BF16>(p0 - f.x, p1 - f.y);
                    // B fragment of step kt for lane (quad = head, tq): b0 = tokens 2tq, 2tq + 1; b1 = the same + 8
                    const int kt = u >> 3, w8 = u & 7;
                    uint32_t* dst = fw + ((size_t)(kt * 32 + warp * 4 + (w8 & 3)) << 2) + (w8 >> 2);
                    dst[0] = hi;                                       // words 0, 1: hi terms
                    dst[2] = lo;                                       // words 2, 3: lo terms
                }
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0 && live) { s_m[warp] = mx; s_l[warp] = sum; }
        }
        __syncthreads();

        // ---- O^T += V^T P^T over the chunk's tiles -----------------------------------------------------------
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        bool ok = true;
        for (int ti = 0; ti < ntiles && ok; ++ti, ++it) {
            const int s = it % LG_STAGES;
            ok = warp_wait(&full[s], (uint32_t)(it / LG_STAGES) & 1u, abort_flag);
            if (!ok) break;
            const uint32_t vbase = tile0 + s * TILE_BYTES;
            if ((ti + 1) * LG_TILE > nt) {
                // Rows past the chunk's last slot hold whatever lies behind it (other slots, NaN patterns).  Every warp
                // clears the part of them that it reads itself - its two 16-byte columns of the rows of its own
                // 16-token steps - so no warp depends on another here (a barrier inside this loop could be left
                // waiting by a warp whose bounded wait ran out).
                for (int u = lane; u < LG_TILE * 2; u += 32) {
                    const int r = u >> 1, cc = 2 * mt + (u & 1);
                    if (ti * LG_TILE + r >= nt && ((r >> 4) % SETS) == set)
                        sts128_zero(vbase + (cc >> 3) * (128u * LG_TILE) + r * 128u + (((cc & 7) ^ (r & 7)) << 4));
                }
                __syncwarp();
            }
#pragma unroll
            for (int k4 = set; k4 < LG_TILE / 16; k4 += SETS) {
                const uint4 f = s_frag[(size_t)(ti * (LG_TILE / 16) + k4) * 32 + lane];
                uint32_t a[4];
                ldmatrix_x4_trans(a, vbase + v_off + (uint32_t)k4 * (16u * 128u));
                mma_16816<BF16>(acc, a, f.x, f.y);
                mma_16816<BF16>(acc, a, f.z, f.w);
            }
            if ((ti + 1) * LG_TILE > nt) fence_proxy_async();          // the cleared rows come before the next TMA write
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
            if (tid == 0 && it + LG_STAGES < total) {
                if (mbar_wait(&empty[s], (uint32_t)(it / LG_STAGES) & 1u, abort_flag)) { issue(it + LG_STAGES); ++issued; }
            }
        }
        // ---- results: acc[0], acc[1]: component 16 mt + quad, heads 2tq, 2tq + 1; acc[2], acc[3]: component + 8 ----
        float* const s_add = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(s_frag) +
                                                      (size_t)((p.chunk + LG_TILE - 1) / LG_TILE * LG_TILE / 16) * 512);
        if constexpr (SETS == 2) {
            if (set == 1) *reinterpret_cast<float4*>(s_add + (mt * 32 + lane) * 4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
        }
        // every warp gets here, whatever became of its waits: the outcome is made uniform at this barrier, so that
        // all warps leave together or none does
        if (!__syncthreads_and(ok ? 1 : 0)) break;
        if constexpr (SETS == 2) {
            if (set == 0) {
                const float4 x = *reinterpret_cast<const float4*>(s_add + (mt * 32 + lane) * 4);
                acc[0] += x.x; acc[1] += x.y; acc[2] += x.z; acc[3] += x.w;
            }
        }
        if (set == 0) {
            const int d = 16 * mt + quad;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int hh = 2 * tq + j;
                if (hh < nh) {
                    const size_t slot = ((size_t)b * p.Hq + h0 + hh) * p.NC + c;
                    const uint64_t keep = l2_evict_last_policy();      // the merge reads these lines next
                    st_global_hint(p.o_part + slot * D + d, acc[j], keep);
                    st_global_hint(p.o_part + slot * D + d + 8, acc[2 + j], keep);
                    if (mt == 0 && quad == 0) { p.m_part[slot] = s_m[hh]; p.l_part[slot] = s_l[hh]; }
                }
            }
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
}

}  // namespace hg
