// Log-sum-exp merge of softmax partials and final normalisation (sm_100a).
//
// One CTA of 8 warps per (sequence, query head) - or, when a row has many partials, a thread-block
// cluster of CLUSTER such CTAs that split the row's partials and combine through distributed shared
// memory.  One sweep: each warp takes every W-th partial (four loads in flight), keeps a running
// maximum M_w and the sums of w_i * o_i and w_i * l_i with w_i = e^{m_i - M_w}, rescaling them when
// M_w grows; each lane holds D/32 contiguous output components.  The warps' triples, then the
// cluster's CTAs' triples, are combined the same way in fixed order, and one division finishes
// out = sum w o / sum w l and lse = M + ln sum w l.  No atomics: bit-reproducible for a given launch
// shape.  A second kernel, one warp per row, serves large batches of short rows.
#pragma once

#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hg {

constexpr int MERGE_MAX_SRC = 8;

// The o rows are read with the hint their producer wrote them with (keep the lines in the L2): partials are scratch
// that the next step overwrites in place, and a line that stays resident is neither written out to DRAM nor
// allocated again.
__device__ __forceinline__ uint64_t merge_keep_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ float4 ld_keep_v4(const float* p, uint64_t pol) {
    float4 v;
    asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ float2 ld_keep_v2(const float* p, uint64_t pol) {
    float2 v;
    asm volatile("ld.global.L2::cache_hint.v2.f32 {%0, %1}, [%2], %3;" : "=f"(v.x), "=f"(v.y) : "l"(p), "l"(pol));
    return v;
}

struct MergeParams {
    const float* o[MERGE_MAX_SRC];
    const float* m[MERGE_MAX_SRC];
    const float* l[MERGE_MAX_SRC];
    int nc[MERGE_MAX_SRC];
    int n_src;
    int total;      // sum of nc
    float* out;
    float* lse;
};

template <int D, int THREADS_, int CLUSTER>
__global__ void __launch_bounds__(THREADS_) merge_kernel(const MergeParams p) {
    namespace cg = cooperative_groups;
    constexpr int VEC = D / 32;
    constexpr int WARPS = THREADS_ / 32;
    __shared__ float s_m[WARPS];
    __shared__ float s_l[WARPS];
    __shared__ float s_o[WARPS][D];
    __shared__ float s_cta_m;                   // this CTA's share, read by its cluster peers
    __shared__ float s_cta_l;
    __shared__ float s_cta_o[D];
    const float NEG_INF = __int_as_float(0xff800000);
    const int row = blockIdx.x / CLUSTER;       // b * Hq + h
    const int rank = blockIdx.x % CLUSTER;      // position in the cluster
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

#if __CUDA_ARCH__ >= 900
    cudaTriggerProgrammaticLaunchCompletion();  // a partial kernel launched as a dependent may set up meanwhile
    cudaGridDependencySynchronize();            // partials may come from the kernel launched just before
#endif
    const uint64_t keep = merge_keep_policy();

    // ---- one sweep: every warp keeps a running maximum and rescales its sums when it grows ----------
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    float lsum = 0.f, Mw = NEG_INF;
    for (int s = 0; s < p.n_src; ++s) {
        const int nc = p.nc[s];
        const float* ms = p.m[s] + (size_t)row * nc;
        const float* ls = p.l[s] + (size_t)row * nc;
        const float* os = p.o[s] + (size_t)row * nc * D;
        for (int i0 = rank * WARPS + warp; i0 < nc; i0 += 4 * CLUSTER * WARPS) {
            float mi[4], li[4], ov[4][VEC];
#pragma unroll
            for (int u = 0; u < 4; ++u) {                      // four independent partials in flight
                const int i = i0 + u * CLUSTER * WARPS;
                const bool in = i < nc;
                mi[u] = in ? ms[i] : NEG_INF;
                li[u] = in ? ls[i] : 0.f;
                const bool live = in && mi[u] != NEG_INF;      // an empty partial's o is not read
                const float* orow = os + (size_t)(in ? i : 0) * D + lane * VEC;
                if constexpr (VEC == 4) {
                    const float4 v = live ? ld_keep_v4(orow, keep) : make_float4(0.f, 0.f, 0.f, 0.f);
                    ov[u][0] = v.x; ov[u][1] = v.y; ov[u][2] = v.z; ov[u][3] = v.w;
                } else {
                    const float2 v = live ? ld_keep_v2(orow, keep) : make_float2(0.f, 0.f);
                    ov[u][0] = v.x; ov[u][1] = v.y;
                }
            }
            const float m4 = fmaxf(fmaxf(mi[0], mi[1]), fmaxf(mi[2], mi[3]));
            if (m4 == NEG_INF) continue;                        // four empty partials (warp-uniform)
            if (m4 > Mw) {
                const float r = __expf(Mw - m4);                // 0 while Mw is still -inf
                lsum *= r;
#pragma unroll
                for (int v = 0; v < VEC; ++v) acc[v] *= r;
                Mw = m4;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float w = mi[u] == NEG_INF ? 0.f : __expf(mi[u] - Mw);
                lsum = fmaf(w, li[u], lsum);
#pragma unroll
                for (int v = 0; v < VEC; ++v) acc[v] = fmaf(w, ov[u][v], acc[v]);
            }
        }
    }
    if (lane == 0) { s_m[warp] = Mw; s_l[warp] = lsum; }
#pragma unroll
    for (int v = 0; v < VEC; ++v) s_o[warp][lane * VEC + v] = acc[v];
    __syncthreads();

    // ---- warps of the CTA, in fixed order ---------------------------------------------------------------
    float M = s_m[0];
#pragma unroll
    for (int w = 1; w < WARPS; ++w) M = fmaxf(M, s_m[w]);
    float Lsum = 0.f, o = 0.f;
    if (tid < D) {
#pragma unroll
        for (int w = 0; w < WARPS; ++w) {
            const float r = s_m[w] == NEG_INF ? 0.f : __expf(s_m[w] - M);
            Lsum = fmaf(r, s_l[w], Lsum);
            o = fmaf(r, s_o[w][tid], o);
        }
    }
    // ---- CTAs of the cluster, in fixed order -------------------------------------------------------------
    if constexpr (CLUSTER > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        if (tid < D) s_cta_o[tid] = o;
        if (tid == 0) { s_cta_l = Lsum; s_cta_m = M; }
        cluster.sync();
        if (rank == 0 && tid < D) {
            float mr[CLUSTER];
#pragma unroll
            for (int r = 0; r < CLUSTER; ++r) mr[r] = *cluster.map_shared_rank(&s_cta_m, r);
            M = mr[0];
#pragma unroll
            for (int r = 1; r < CLUSTER; ++r) M = fmaxf(M, mr[r]);
            Lsum = 0.f; o = 0.f;
#pragma unroll
            for (int r = 0; r < CLUSTER; ++r) {
                const float w = mr[r] == NEG_INF ? 0.f : __expf(mr[r] - M);
                Lsum = fmaf(w, *cluster.map_shared_rank(&s_cta_l, r), Lsum);
                o = fmaf(w, cluster.map_shared_rank(&s_cta_o[0], r)[tid], o);
            }
        }
        cluster.sync();                         // peers keep their shared memory alive until rank 0 has read it
        if (rank != 0) return;
    }
    if (tid < D) {
        const bool empty = (M == NEG_INF);
        p.out[(size_t)row * D + tid] = empty ? 0.f : o / Lsum;
        if (tid == 0 && p.lse) p.lse[row] = empty ? NEG_INF : M + logf(Lsum);
    }
}

// Many rows (a large batch): one WARP per (sequence, query head), eight rows per CTA.  The warp reads 32 slot
// maxima at a time, one per lane, and visits only the slots that hold something, in order, four loads in flight -
// so the many empty slots that short sequences have next to a long one cost almost nothing.  Same
// running-maximum rule as above; no shared memory, no barrier.
template <int D>
__global__ void __launch_bounds__(256) merge_rows_kernel(const MergeParams p, int rows) {
    constexpr int VEC = D / 32;
    const float NEG_INF = __int_as_float(0xff800000);
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
#if __CUDA_ARCH__ >= 900
    cudaTriggerProgrammaticLaunchCompletion();  // a partial kernel launched as a dependent may set up meanwhile
    cudaGridDependencySynchronize();
#endif
    if (row >= rows) return;
    const uint64_t keep = merge_keep_policy();
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    float lsum = 0.f, M = NEG_INF;
    for (int s = 0; s < p.n_src; ++s) {
        const int nc = p.nc[s];
        const float* ms = p.m[s] + (size_t)row * nc;
        const float* ls = p.l[s] + (size_t)row * nc;
        const float* os = p.o[s] + (size_t)row * nc * D;
        for (int i0 = 0; i0 < nc; i0 += 32) {
            const float mine = i0 + lane < nc ? ms[i0 + lane] : NEG_INF;
            uint32_t live = __ballot_sync(0xffffffffu, mine != NEG_INF);
            while (live) {
                float mi[4], li[4], ov[4][VEC];
#pragma unroll
                for (int u = 0; u < 4; ++u) {                  // the next four live slots (warp-uniform)
                    const bool in = live != 0u;
                    const int src = in ? __ffs(live) - 1 : 0;
                    if (in) live &= live - 1u;
                    mi[u] = __shfl_sync(0xffffffffu, mine, src);
                    if (!in) mi[u] = NEG_INF;
                    const int i = i0 + src;
                    li[u] = in ? ls[i] : 0.f;
                    const float* orow = os + (size_t)i * D + lane * VEC;
                    if constexpr (VEC == 4) {
                        const float4 v = in ? ld_keep_v4(orow, keep) : make_float4(0.f, 0.f, 0.f, 0.f);
                        ov[u][0] = v.x; ov[u][1] = v.y; ov[u][2] = v.z; ov[u][3] = v.w;
                    } else {
                        const float2 v = in ? ld_keep_v2(orow, keep) : make_float2(0.f, 0.f);
                        ov[u][0] = v.x; ov[u][1] = v.y;
                    }
                }
                const float m4 = fmaxf(fmaxf(mi[0], mi[1]), fmaxf(mi[2], mi[3]));
                if (m4 > M) {
                    const float r = __expf(M - m4);            // 0 while M is still -inf
                    lsum *= r;
#pragma unroll
                    for (int v = 0; v < VEC; ++v) acc[v] *= r;
                    M = m4;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float w = mi[u] == NEG_INF ? 0.f : __expf(mi[u] - M);
                    lsum = fmaf(w, li[u], lsum);
#pragma unroll
                    for (int v = 0; v < VEC; ++v) acc[v] = fmaf(w, ov[u][v], acc[v]);
                }
            }
        }
    }
    const bool empty = (M == NEG_INF);
    float* out = p.out + (size_t)row * D + lane * VEC;
#pragma unroll
    for (int v = 0; v < VEC; ++v) out[v] = empty ? 0.f : acc[v] / lsum;
    if (lane == 0 && p.lse) p.lse[row] = empty ? NEG_INF : M + logf(lsum);
}

}  // namespace hg
