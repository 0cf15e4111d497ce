/*
 * The C ABI used from plain C: no Python, no torch.  Builds a small paged problem in host memory, copies it
 * to the device with the CUDA runtime, calls hg_attn_workspace_bytes + hg_attn_decode, and compares out / lse
 * with the fp64 oracle (linked in as test infrastructure).  Exit code 0 and a line "C ABI parity OK" on success.
 *
 * Layout: contiguous cache (block_table = NULL), rows [page][token][head][D], so that sequence b's tokens are
 * the oracle's logical cache [B][Lmax][Hkv][D] with Lmax = max_pages * page_size - one buffer serves both.
 */
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "hybridgen_attn.h"

void hgo_full_batch(const uint16_t* q, const uint16_t* K, const uint16_t* V, int B, int Hq, int Hkv, int D, int dtype,
                    int64_t Lmax, double scale, const int64_t* lo, const int64_t* hi, double* out, double* lse, int threads);

#define CHECK_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_)); return 2; } } while (0)
#define CHECK_HG(x) do { hg_status s_ = (x); if (s_ != HG_OK) { fprintf(stderr, "%s: %s\n", #x, hg_status_string(s_)); return 3; } } while (0)

/* binary16 pattern of k / 32 for |k| <= 2048: exactly representable, so no rounding rule is involved */
static uint16_t half_of_32nds(int k) {
    if (k == 0) return 0;
    const uint16_t sign = k < 0 ? 0x8000u : 0;
    unsigned a = (unsigned)abs(k);
    int e = 0;
    while ((a >> (e + 1)) != 0) ++e;            /* a = 1.xxx * 2^e */
    const int exp = e - 5 + 15;                 /* value = a / 32 */
    const unsigned man = ((a << (10 - e)) & 0x3ffu);
    return (uint16_t)(sign | (unsigned)(exp << 10) | man);
}

static uint32_t lcg(uint32_t* s) { *s = *s * 1664525u + 1013904223u; return *s >> 8; }

int main(void) {
    enum { B = 2, HQ = 8, HKV = 2, D = 64, PAGE = 16, MAXP = 24, LMAX = PAGE * MAXP, C = 128, NC = 3 };
    const int32_t seq_lens[B] = {371, 150}, tok_begin[B] = {37, 0}, tok_end[B] = {371, 150};
    const size_t kv_elems = (size_t)B * LMAX * HKV * D, q_elems = (size_t)B * HQ * D;
    uint16_t* hk = malloc(kv_elems * 2); uint16_t* hv = malloc(kv_elems * 2); uint16_t* hq = malloc(q_elems * 2);
    uint32_t seed = 12345u;
    for (size_t i = 0; i < kv_elems; ++i) { hk[i] = half_of_32nds((int)(lcg(&seed) % 129u) - 64); hv[i] = half_of_32nds((int)(lcg(&seed) % 257u) - 128); }
    for (size_t i = 0; i < q_elems; ++i) hq[i] = half_of_32nds((int)(lcg(&seed) % 65u) - 32);

    /* oracle: monolithic attention over [tok_begin, tok_end) */
    const int64_t lo[B] = {tok_begin[0], tok_begin[1]}, hi[B] = {tok_end[0], tok_end[1]};
    double* ref_out = malloc(sizeof(double) * B * HQ * D); double ref_lse[B * HQ];
    hgo_full_batch(hq, hk, hv, B, HQ, HKV, D, /*f16*/ 0, LMAX, 0.0, lo, hi, ref_out, ref_lse, 2);

    /* device side through the C ABI */
    void *dk, *dv, *dq, *ws; int32_t *dsl, *dtb, *dte, *dstatus; float *dout, *dlse;
    CHECK_CUDA(cudaMalloc(&dk, kv_elems * 2)); CHECK_CUDA(cudaMalloc(&dv, kv_elems * 2)); CHECK_CUDA(cudaMalloc(&dq, q_elems * 2));
    CHECK_CUDA(cudaMalloc((void**)&dsl, sizeof seq_lens)); CHECK_CUDA(cudaMalloc((void**)&dtb, sizeof tok_begin));
    CHECK_CUDA(cudaMalloc((void**)&dte, sizeof tok_end)); CHECK_CUDA(cudaMalloc((void**)&dstatus, 4));
    CHECK_CUDA(cudaMalloc((void**)&dout, sizeof(float) * B * HQ * D)); CHECK_CUDA(cudaMalloc((void**)&dlse, sizeof(float) * B * HQ));
    CHECK_CUDA(cudaMemcpy(dk, hk, kv_elems * 2, cudaMemcpyHostToDevice)); CHECK_CUDA(cudaMemcpy(dv, hv, kv_elems * 2, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(dq, hq, q_elems * 2, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(dsl, seq_lens, sizeof seq_lens, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(dtb, tok_begin, sizeof tok_begin, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(dte, tok_end, sizeof tok_end, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemset(dstatus, 0, 4));

    hg_attn_desc d;
    memset(&d, 0, sizeof d);
    d.struct_size = sizeof d;
    d.batch = B; d.num_q_heads = HQ; d.num_kv_heads = HKV; d.head_dim = D; d.dtype = HG_DTYPE_F16;
    d.page_size = PAGE; d.num_pages = B * MAXP; d.max_pages = MAXP;
    d.tok_stride = HKV * D; d.head_stride = D; d.page_stride = (int64_t)PAGE * HKV * D;
    d.block_table = NULL; d.chunk_tokens = C; d.num_chunks = NC; d.scale = 0.f; d.status = dstatus;
    const size_t ws_bytes = hg_attn_workspace_bytes(&d, 0);
    if (ws_bytes == 0) { fprintf(stderr, "workspace_bytes rejected the description\n"); return 4; }
    CHECK_CUDA(cudaMalloc(&ws, ws_bytes));
    cudaStream_t stream;
    CHECK_CUDA(cudaStreamCreate(&stream));
    CHECK_HG(hg_attn_decode(dq, dk, dv, dsl, dtb, dte, NULL, 0, dout, dlse, ws, ws_bytes, stream, &d));
    CHECK_CUDA(cudaStreamSynchronize(stream));
    float* out = malloc(sizeof(float) * B * HQ * D); float lse[B * HQ]; int32_t status = -1;
    CHECK_CUDA(cudaMemcpy(out, dout, sizeof(float) * B * HQ * D, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(lse, dlse, sizeof lse, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(&status, dstatus, 4, cudaMemcpyDeviceToHost));
    if (status != HG_DEV_OK) { fprintf(stderr, "device status %d\n", status); return 5; }

    double max_abs = 0, num = 0, den = 0, lse_abs = 0;
    for (int i = 0; i < B * HQ * D; ++i) {
        const double e = fabs((double)out[i] - ref_out[i]);
        if (!(e <= max_abs)) max_abs = e;       /* a NaN would stick */
        num += e * e; den += ref_out[i] * ref_out[i];
    }
    for (int i = 0; i < B * HQ; ++i) { const double e = fabs((double)lse[i] - ref_lse[i]); if (!(e <= lse_abs)) lse_abs = e; }
    const double rel = sqrt(num / den);
    printf("out max_abs %.3e rel_l2 %.3e lse_abs %.3e\n", max_abs, rel, lse_abs);
    if (!(max_abs <= 2e-3) || !(rel <= 1e-3) || !(lse_abs <= 1e-4)) { fprintf(stderr, "parity FAILED\n"); return 1; }
    printf("C ABI parity OK (version %u)\n", hg_version());
    return 0;
}
