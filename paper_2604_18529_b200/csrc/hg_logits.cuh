// Softmax partial from host-computed logits and gathered V rows (sm_100a): the device side of the
// paper's CPU -> GPU hand-off.  The host ships, per (sequence, query head), the scaled logits of its
// selected tokens and, per (sequence, KV head), the matching V rows; this kernel turns every chunk of
// them into the same (m, l, o) partial that hg_attn_partial produces for GPU-resident tokens, so the
// merge kernel treats both sides alike.  q.K^T is skipped; only V is streamed.
//
// Grid (chunk, KV head, sequence), 256 threads.  Per block of up to NH (1, 2, 4 or 8) query heads of the group: the
// chunk's logits go to shared memory, warp h finds head h's maximum and turns its logits into
// p = e^{s - m} in place (and their sum l); then the 8 warps stride over the chunk's tokens, each lane
// owning D/32 components of every head's o, reading each V row once for all heads; a fixed-order
// cross-warp sum finishes.  fp32 throughout, no atomics.
#pragma once

#include "hg_device.cuh"

namespace hg {

constexpr int LG_THREADS = 256;
constexpr int LG_WARPS = LG_THREADS / 32;
constexpr int LG_MAX_CHUNK = 1024;    // selected tokens per chunk

struct LogitsParams {
    const float* logits;      // [B][Hq][K]
    const void* v_rows;       // [B][Hkv][K][D]
    const int32_t* n_sel;     // [B]
    float* o_part;            // [B][Hq][NC][D]
    float* m_part;            // [B][Hq][NC]
    float* l_part;
    int B, Hq, Hkv, G, K, chunk, NC;
};

// NH: query heads handled per pass over the chunk's V rows (1, 2, 4 or 8; a group of G heads takes ceil(G / NH) passes)
template <int D, bool BF16, int NH>
__global__ void __launch_bounds__(LG_THREADS) logits_partial_kernel(const LogitsParams p) {
    constexpr int VEC = D / 32;                       // components per lane
    extern __shared__ float lg_smem[];
    float* const s_p = lg_smem;                       // [NH heads][chunk]  logits, then p
    float* const s_red = lg_smem + NH * p.chunk;      // [8 warps][NH heads][D]
    __shared__ float s_m[NH], s_l[NH];
    const float NEG_INF = __int_as_float(0xff800000);

    const int c = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = min(max(p.n_sel[b], 0), p.K);
    const int t0 = c * p.chunk, t1 = min(t0 + p.chunk, n);
    const int nt = max(t1 - t0, 0);
    const uint16_t* vbase = reinterpret_cast<const uint16_t*>(p.v_rows) + ((size_t)b * p.Hkv + g) * (size_t)p.K * D;

    for (int hb = 0; hb * NH < p.G; ++hb) {
        const int h0 = g * p.G + hb * NH, nh = min(NH, p.G - hb * NH);
        // ---- logits of this head block into shared memory -------------------------------------------
        for (int i = tid; i < nh * nt; i += LG_THREADS) {
            const int hh = i / nt, t = i - hh * nt;
            s_p[hh * p.chunk + t] = p.logits[((size_t)b * p.Hq + h0 + hh) * p.K + t0 + t];
        }
        __syncthreads();
        // ---- warp h: maximum of head h, p = e^{s - m} in place, l = sum p ------------------------------
        if (warp < nh) {
            float* row = s_p + warp * p.chunk;
            float mx = NEG_INF;
            for (int t = lane; t < nt; t += 32) mx = fmaxf(mx, row[t]);
#pragma unroll
            for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float sum = 0.f;
            for (int t = lane; t < nt; t += 32) {
                const float pv = (mx == NEG_INF) ? 0.f : __expf(row[t] - mx);
                row[t] = pv;
                sum += pv;
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) { s_m[warp] = mx; s_l[warp] = sum; }
        }
        __syncthreads();
        // ---- o[h][d] = sum_t p[h][t] V[t][d]: each V row read once for all heads of the block -----------
        float acc[NH][VEC];
#pragma unroll
        for (int hh = 0; hh < NH; ++hh)
#pragma unroll
            for (int v = 0; v < VEC; ++v) acc[hh][v] = 0.f;
        constexpr int UNROLL = 8;                                  // V rows in flight per warp
        for (int tt = warp; tt < nt; tt += UNROLL * LG_WARPS) {
            uint2 raw[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int t = tt + u * LG_WARPS;
                raw[u] = make_uint2(0u, 0u);
                if (t < nt) {
                    const uint16_t* vrow = vbase + (size_t)(t0 + t) * D + lane * VEC;
                    if constexpr (VEC == 4) raw[u] = *reinterpret_cast<const uint2*>(vrow);
                    else raw[u].x = *reinterpret_cast<const uint32_t*>(vrow);
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int t = tt + u * LG_WARPS;
                if (t >= nt) break;
                float vv[VEC];
                const float2 a = unpack2<BF16>(raw[u].x);
                vv[0] = a.x; vv[1] = a.y;
                if constexpr (VEC == 4) {
                    const float2 bb = unpack2<BF16>(raw[u].y);
                    vv[2] = bb.x; vv[3] = bb.y;
                }
#pragma unroll
                for (int hh = 0; hh < NH; ++hh) {
                    if (NH == 1 || hh < nh) {
                        const float pv = s_p[hh * p.chunk + t];       // broadcast read
                        if (pv != 0.f) {                              // unselected slots (and their V rows) never enter the sum
#pragma unroll
                            for (int v = 0; v < VEC; ++v) acc[hh][v] = fmaf(pv, vv[v], acc[hh][v]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) {
            if (NH == 1 || hh < nh) {
#pragma unroll
                for (int v = 0; v < VEC; ++v) s_red[((size_t)warp * NH + hh) * D + lane * VEC + v] = acc[hh][v];
            }
        }
        __syncthreads();
        for (int i = tid; i < nh * D; i += LG_THREADS) {
            const int hh = i / D, d = i - hh * D;
            float o = 0.f;
#pragma unroll
            for (int w = 0; w < LG_WARPS; ++w) o += s_red[((size_t)w * NH + hh) * D + d];
            const size_t slot = ((size_t)b * p.Hq + h0 + hh) * p.NC + c;
            p.o_part[slot * D + d] = o;
            if (d == 0) { p.m_part[slot] = s_m[hh]; p.l_part[slot] = s_l[hh]; }
        }
        __syncthreads();
    }
}

}  // namespace hg
