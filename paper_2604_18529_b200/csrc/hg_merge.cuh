// Log-sum-exp merge of softmax partials and final normalisation (sm_100a).
//
// One CTA per (sequence, query head), 8 or 32 warps depending on how many partials a row has.  Pass 1
// finds M = max_i m_i over every partial of every source; pass 2 accumulates w_i * o_i and w_i * l_i
// with w_i = e^{m_i - M}, each warp taking every W-th partial (four loads in flight) and each lane D/32
// contiguous output components; a fixed-order cross-warp sum and one division finish
// out = sum w o / sum w l and lse = M + ln sum w l.  No atomics: bit-reproducible.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace hg {

constexpr int MERGE_MAX_SRC = 8;

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

template <int D, int THREADS_>
__global__ void __launch_bounds__(THREADS_) merge_kernel(const MergeParams p) {
    constexpr int VEC = D / 32;
    constexpr int WARPS = THREADS_ / 32;
    __shared__ float s_max[WARPS];
    __shared__ float s_l[WARPS];
    __shared__ float s_o[WARPS][D];
    const float NEG_INF = __int_as_float(0xff800000);
    const int row = blockIdx.x;                 // b * Hq + h
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

#if __CUDA_ARCH__ >= 900
    cudaGridDependencySynchronize();            // partials may come from the kernel launched just before
#endif

    // ---- pass 1: global maximum -------------------------------------------------------------------
    float mx = NEG_INF;
    for (int s = 0; s < p.n_src; ++s) {
        const float* ms = p.m[s] + (size_t)row * p.nc[s];
        for (int i = tid; i < p.nc[s]; i += THREADS_) mx = fmaxf(mx, ms[i]);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) s_max[warp] = mx;
    __syncthreads();
    float M = s_max[0];
#pragma unroll
    for (int w = 1; w < WARPS; ++w) M = fmaxf(M, s_max[w]);

    // ---- pass 2: weighted sums ----------------------------------------------------------------------
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    float lsum = 0.f;
    if (M != NEG_INF) {
        for (int s = 0; s < p.n_src; ++s) {
            const int nc = p.nc[s];
            const float* ms = p.m[s] + (size_t)row * nc;
            const float* ls = p.l[s] + (size_t)row * nc;
            const float* os = p.o[s] + (size_t)row * nc * D;
            for (int i0 = warp; i0 < nc; i0 += 4 * WARPS) {
                float mi[4], li[4], ov[4][VEC];
#pragma unroll
                for (int u = 0; u < 4; ++u) {                  // four independent partials in flight
                    const int i = i0 + u * WARPS;
                    const bool in = i < nc;
                    mi[u] = in ? ms[i] : NEG_INF;
                    li[u] = in ? ls[i] : 0.f;
                    const bool live = in && mi[u] != NEG_INF;  // an empty partial's o is not read
                    const float* orow = os + (size_t)(in ? i : 0) * D + lane * VEC;
                    if constexpr (VEC == 4) {
                        const float4 v = live ? *reinterpret_cast<const float4*>(orow) : make_float4(0.f, 0.f, 0.f, 0.f);
                        ov[u][0] = v.x; ov[u][1] = v.y; ov[u][2] = v.z; ov[u][3] = v.w;
                    } else {
                        const float2 v = live ? *reinterpret_cast<const float2*>(orow) : make_float2(0.f, 0.f);
                        ov[u][0] = v.x; ov[u][1] = v.y;
                    }
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
    if (lane == 0) s_l[warp] = lsum;
#pragma unroll
    for (int v = 0; v < VEC; ++v) s_o[warp][lane * VEC + v] = acc[v];
    __syncthreads();

    if (tid < D) {
        float Lsum = 0.f, o = 0.f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) { Lsum += s_l[w]; o += s_o[w][tid]; }
        const bool empty = (M == NEG_INF);
        p.out[(size_t)row * D + tid] = empty ? 0.f : o / Lsum;
        if (tid == 0 && p.lse) p.lse[row] = empty ? NEG_INF : M + logf(Lsum);
    }
}

}  // namespace hg
