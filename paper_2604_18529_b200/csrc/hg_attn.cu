// Host side of the C ABI declared in include/hybridgen_attn.h: argument validation, TMA tensor-map
// encoding, launches.  No allocation, no synchronisation, no global mutable state (the cached
// driver entry point, the per-kernel shared-memory opt-in and the per-device address of the static
// scratch array are idempotent).
#include "hybridgen_attn.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stddef.h>
#ifdef HG_TRACE
#include <stdlib.h>
#endif
#include <string.h>

#include <atomic>

#include "hg_kvcache.cuh"
#include "hg_logits.cuh"
#include "hg_logits_tc.cuh"
#include "hg_merge.cuh"
#include "hg_partial.cuh"
#include "hg_stage.cuh"

namespace hg {

constexpr int kMaxDevices = 64;

// ---- validation ------------------------------------------------------------------------------------

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The optional trailing field, for callers compiled against a shorter struct.
static int32_t* desc_sched(const hg_attn_desc* d) {
    return d->struct_size >= offsetof(hg_attn_desc, sched_counter) + sizeof(int32_t*) ? d->sched_counter : nullptr;
}

// Multiplier and shift that divide a number below 2^31 by d (see FastDiv).
static FastDiv make_fast_div(uint32_t d) {
    FastDiv f = {0u, 0u};
    if (d <= 1) return f;
    uint32_t s = 0;
    while ((1ull << s) < d) ++s;                                   // ceil(log2 d) >= 1
    f.mul = (uint32_t)(((1ull << (31 + s)) + d - 1) / d);          // < 2^32 because d > 2^(s-1)
    f.shift = s - 1;
    return f;
}

static int ilog2_exact(int v) {
    for (int s = 0; s < 31; ++s)
        if ((1 << s) == v) return s;
    return -1;
}

// Checks the fields every entry point relies on.  `need_kv` also checks the KV addressing.
static hg_status check_desc(const hg_attn_desc* d, bool need_kv) {
    if (!d || d->struct_size < offsetof(hg_attn_desc, sched_counter)) return HG_ERR_INVALID_ARG;
    if (d->batch < 1 || d->batch > 65535) return HG_ERR_INVALID_ARG;
    if (d->num_kv_heads < 1 || d->num_q_heads < 1 || d->num_q_heads % d->num_kv_heads) return HG_ERR_INVALID_ARG;
    if (d->head_dim <= 0 || d->head_dim % 8) return HG_ERR_INVALID_ARG;
    if (d->head_dim != 64 && d->head_dim != 128) return HG_ERR_UNSUPPORTED;
    if (!need_kv) return HG_OK;
    if (d->dtype != HG_DTYPE_F16 && d->dtype != HG_DTYPE_BF16) return HG_ERR_INVALID_ARG;
    if (d->page_size < 1 || d->num_pages < 1 || d->max_pages < 1) return HG_ERR_INVALID_ARG;
    if (d->page_stride < 0 || d->head_stride < 0 || d->tok_stride < d->head_dim) return HG_ERR_INVALID_ARG;
    if ((d->page_stride | d->head_stride | d->tok_stride) & 7) return HG_ERR_INVALID_ARG;   // 16-byte multiples
    if (d->chunk_tokens < 1 || d->num_chunks < 1) return HG_ERR_INVALID_ARG;
    if (!(d->scale >= 0.f) || isinf(d->scale)) return HG_ERR_INVALID_ARG;
    const int shift = ilog2_exact(d->page_size);
    if (shift < 4 || shift > 8) return HG_ERR_UNSUPPORTED;                                   // 16 .. 256
    if (d->chunk_tokens % TILE_T || d->chunk_tokens % d->page_size || d->chunk_tokens > 65536)
        return HG_ERR_UNSUPPORTED;
    if (d->chunk_tokens / d->page_size > MAX_CHUNK_PAGES) return HG_ERR_UNSUPPORTED;
    if (desc_sched(d) && (reinterpret_cast<uintptr_t>(desc_sched(d)) & 7u)) return HG_ERR_INVALID_ARG;
    if ((int64_t)d->num_kv_heads * ((d->num_q_heads / d->num_kv_heads + 7) / 8) > 65535) return HG_ERR_UNSUPPORTED;
    if (!d->block_table && (int64_t)d->batch * d->max_pages > d->num_pages) return HG_ERR_INVALID_ARG;
    return HG_OK;
}

// ---- tensor maps -------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &f, 12000, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// Pool viewed as a 5-D tensor {d within a 64-element half, token in page, half, head, page}; one box is a
// whole page of one head: [half][rows][64 elements = 128 bytes, swizzled].  The half dimension sits
// behind the token dimension (its stride, 128 bytes, is the smaller one) so that the box lands in
// shared memory as two 128-byte-wide column blocks, the layout ldmatrix reads without bank conflicts.
static hg_status make_maps(const hg_attn_desc* d, const void* k, const void* v, CUtensorMap* tk, CUtensorMap* tv) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return HG_ERR_CUDA;
    const int rows = d->page_size >= TILE_T ? TILE_T : d->page_size;
    const int halves = d->head_dim / 64;
    cuuint64_t dims[5] = {64, (cuuint64_t)d->page_size, (cuuint64_t)halves, (cuuint64_t)d->num_kv_heads,
                          (cuuint64_t)d->num_pages};
    cuuint64_t strides[4] = {(cuuint64_t)d->tok_stride * 2u, 128u, (cuuint64_t)d->head_stride * 2u,
                             (cuuint64_t)d->page_stride * 2u};
    if (d->num_kv_heads == 1) strides[2] = strides[0];     // unused dimensions still need a legal stride
    if (d->num_pages == 1) strides[3] = strides[0];
    cuuint32_t box[5] = {64, (cuuint32_t)rows, (cuuint32_t)halves, 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    const CUtensorMapDataType dt = d->dtype == HG_DTYPE_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    const void* base[2] = {k, v};
    CUtensorMap* out[2] = {tk, tv};
    for (int i = 0; i < 2; ++i) {
        CUresult r = enc(out[i], dt, 5, const_cast<void*>(base[i]), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return HG_ERR_UNSUPPORTED;   // a stride pattern the TMA unit cannot express
    }
    return HG_OK;
}

// ---- launches ---------------------------------------------------------------------------------------

// The optional tuning fields (all defaults when the caller's struct ends before them).
struct Tune {
    uint32_t bits;
    int stages, ctas_per_sm;
    bool off(uint32_t bit) const { return (bits & bit) != 0; }
};

static Tune desc_tune(const hg_attn_desc* d) {
    Tune t = {0u, 0, 0};
    if (d->struct_size >= offsetof(hg_attn_desc, tune_ctas_per_sm) + sizeof(int32_t)) {
        t.bits = d->tune; t.stages = d->tune_stages; t.ctas_per_sm = d->tune_ctas_per_sm;
    }
    return t;
}

// Per kernel instantiation and device: the shared-memory opt-in that is in force and the occupancy it gives.
// Looked up once per (device, size); racing threads would store the same values.
struct LaunchCache {
    std::atomic<int> smem[kMaxDevices];
    std::atomic<int> per_sm[kMaxDevices];
    std::atomic<int> sms[kMaxDevices];
};

template <int D, bool BF16, int MODE>
static hg_status launch_partial_t(const CUtensorMap& tk, const CUtensorMap& tv, PartialParams p, cudaStream_t st,
                                  bool counter_is_zero, const Tune& tune) {
    static LaunchCache cache;                     // zero-initialised
    const size_t smem = (size_t)p.stages * ((128 / D) * 2 * TILE_T * D * 2 + 8 * D * 2) + 1024;   // per stage: 128 / D x (K tile, V tile), q rows
    auto kern = partial_kernel<D, BF16, MODE>;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return HG_ERR_CUDA; }
    if (cache.smem[dev].load(std::memory_order_acquire) != (int)smem) {
        int sms = 0, per_sm = 0;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, THREADS, smem) != cudaSuccess || per_sm < 1) {
            cudaGetLastError();
            return HG_ERR_CUDA;
        }
        cache.sms[dev].store(sms, std::memory_order_relaxed);
        cache.per_sm[dev].store(per_sm, std::memory_order_relaxed);
        cache.smem[dev].store((int)smem, std::memory_order_release);
    }
    const int Y = p.Hkv * p.head_blocks;
    dim3 grid((unsigned)p.NC, (unsigned)Y, (unsigned)p.B);
    if (p.persistent) {
        // one wave of resident CTAs; each takes items from the schedule
        int per_sm = cache.per_sm[dev].load(std::memory_order_relaxed);
        if (tune.ctas_per_sm >= 1 && tune.ctas_per_sm < per_sm) per_sm = tune.ctas_per_sm;
        const long long slots = (long long)p.NC * Y * p.B;
        const long long resident = (long long)cache.sms[dev].load(std::memory_order_relaxed) * per_sm;
        grid = dim3((unsigned)(slots < resident ? slots : resident), 1, 1);
        if (slots <= resident) p.sched = nullptr;     // at most one item per CTA: nothing to hand out, no counter to clear
    }
    if (p.sched && !counter_is_zero && cudaMemsetAsync(p.sched, 0, 2 * sizeof(int32_t), st) != cudaSuccess) {
        cudaGetLastError();
        return HG_ERR_CUDA;
    }
    if ((!p.sched || counter_is_zero) && !tune.off(HG_TUNE_NO_PDL)) {
        // no memset sits between this launch and the kernel before it in the stream: launch as a programmatic
        // dependent, so that block scheduling and the input-free part of the set-up overlap that kernel's tail
        p.pdl_wait = 1;
        p.spec_prefetch = tune.off(HG_TUNE_NO_SPEC_PREFETCH) ? 0 : 6;
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = grid; cfg.blockDim = dim3(THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, kern, tk, tv, p) != cudaSuccess) { cudaGetLastError(); return HG_ERR_CUDA; }
        return HG_OK;
    }
    kern<<<grid, THREADS, smem, st>>>(tk, tv, p);
    return cudaGetLastError() == cudaSuccess ? HG_OK : HG_ERR_CUDA;
}

template <int MODE>
static hg_status launch_partial_m(int D, bool bf16, const CUtensorMap& tk, const CUtensorMap& tv, const PartialParams& p,
                                  cudaStream_t st, bool counter_is_zero, const Tune& tune) {
    if (D == 128)
        return bf16 ? launch_partial_t<128, true, MODE>(tk, tv, p, st, counter_is_zero, tune)
                    : launch_partial_t<128, false, MODE>(tk, tv, p, st, counter_is_zero, tune);
    return bf16 ? launch_partial_t<64, true, MODE>(tk, tv, p, st, counter_is_zero, tune)
                : launch_partial_t<64, false, MODE>(tk, tv, p, st, counter_is_zero, tune);
}

static hg_status run_partial(int mode, const void* q, const void* k, const void* v, const int32_t* seq_lens,
                             const int32_t* tok_begin, const int32_t* tok_end, float* o_part, float* m_part, float* l_part,
                             uint32_t* sink, void* stream, const hg_attn_desc* d, bool counter_is_zero = false) {
    hg_status st = check_desc(d, true);
    if (st != HG_OK) return st;
    if (!k || !v || !seq_lens || !tok_begin || !tok_end) return HG_ERR_INVALID_ARG;
    if (d->flags & HG_FLAG_COUNTER_CLEAN) counter_is_zero = true;      // the caller vouches for it
    if (mode == MODE_PROBE) {
        if (!sink) return HG_ERR_INVALID_ARG;
    } else if (!q || !o_part || !m_part || !l_part) {
        return HG_ERR_INVALID_ARG;
    }
    if (!aligned16(k) || !aligned16(v) || (q && !aligned16(q)) || (o_part && !aligned16(o_part))) return HG_ERR_INVALID_ARG;

    PartialParams p;
    memset(&p, 0, sizeof p);
    CUtensorMap tk, tv;
    st = make_maps(d, k, v, &tk, &tv);
    if (st != HG_OK) return st;
    const int G = d->num_q_heads / d->num_kv_heads;
    const Tune tune = desc_tune(d);
    // groups of up to 8 query heads: one MMA head block per item; larger groups: items of 16 heads (two blocks)
    if (mode != MODE_PROBE) mode = (G == 1) ? MODE_MHA : (G <= 8 || tune.off(HG_TUNE_NO_GQA16) ? MODE_GQA : MODE_GQA2);
    p.q = q; p.seq_lens = seq_lens; p.tok_begin = tok_begin; p.tok_end = tok_end; p.block_table = d->block_table;
    p.o_part = o_part; p.m_part = m_part; p.l_part = l_part; p.sink = sink; p.status = d->status;
    p.B = d->batch; p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.G = G;
    p.page_size = d->page_size; p.page_shift = ilog2_exact(d->page_size); p.max_pages = d->max_pages;
    p.num_pages = d->num_pages; p.C = d->chunk_tokens; p.NC = d->num_chunks;
    p.head_blocks = (mode == MODE_GQA) ? (G + 7) / 8 : (mode == MODE_GQA2 ? (G + 15) / 16 : 1);
    p.div_C = make_fast_div((uint32_t)p.C);
    p.div_Hkv = make_fast_div((uint32_t)p.Hkv);
    const float scale = d->scale > 0.f ? d->scale : 1.0f / sqrtf((float)d->head_dim);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.stages = tune.stages >= 2 ? (tune.stages > MAX_STAGES ? MAX_STAGES : tune.stages) : 3;   // 3 x 32 KB of K and V (plus q rows): 2 CTAs per SM
    // persistent schedule unless the batch or the chunk's page list exceeds what the kernel keeps in shared memory
    p.persistent = (d->batch <= PERSIST_MAX_BATCH && d->chunk_tokens / d->page_size <= PERSIST_CHUNK_PAGES)
                       ? (tune.off(HG_TUNE_NO_PERSISTENT) ? 0 : 1) : 0;
    p.test_stall = (d->flags & HG_FLAG_TEST_STALL) ? 1 : 0;
    p.sparse_empty = (d->flags & HG_FLAG_SPARSE_EMPTY) ? 1 : 0;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    p.sched = p.persistent && !tune.off(HG_TUNE_NO_DYNAMIC) ? desc_sched(d) : nullptr;
#ifdef HG_TRACE
    { const char* e = getenv("HG_TRACE_PTR"); p.trace = e ? reinterpret_cast<long long*>(strtoull(e, nullptr, 16)) : nullptr; }
#endif
    const bool bf16 = d->dtype == HG_DTYPE_BF16;
    switch (mode) {
        case MODE_MHA: return launch_partial_m<MODE_MHA>(d->head_dim, bf16, tk, tv, p, cs, counter_is_zero, tune);
        case MODE_GQA: return launch_partial_m<MODE_GQA>(d->head_dim, bf16, tk, tv, p, cs, counter_is_zero, tune);
        case MODE_GQA2: return launch_partial_m<MODE_GQA2>(d->head_dim, bf16, tk, tv, p, cs, counter_is_zero, tune);
        default: return launch_partial_m<MODE_PROBE>(d->head_dim, bf16, tk, tv, p, cs, counter_is_zero, tune);
    }
}

static hg_status run_merge(const hg_partial_src* src, int32_t n_src, float* out, float* lse, void* stream,
                           const hg_attn_desc* d) {
    hg_status st = check_desc(d, false);
    if (st != HG_OK) return st;
    if (!src || n_src < 1 || n_src > HG_MAX_MERGE_SRC || !out) return HG_ERR_INVALID_ARG;
    MergeParams p;
    memset(&p, 0, sizeof p);
    for (int i = 0; i < n_src; ++i) {
        if (!src[i].o || !src[i].m || !src[i].l || src[i].nc < 1) return HG_ERR_INVALID_ARG;
        if (!aligned16(src[i].o)) return HG_ERR_INVALID_ARG;
        p.o[i] = src[i].o; p.m[i] = src[i].m; p.l[i] = src[i].l; p.nc[i] = src[i].nc;
        p.total += src[i].nc;
    }
    p.n_src = n_src; p.out = out; p.lse = lse;

    // long rows and few of them: a cluster of 2, 4 or 8 CTAs splits each row's partials, as long as the grid
    // stays within about 256 CTAs (64 rows of 548 partials: 256 CTAs 1.2 us per step ahead of 512, 2.8 us ahead of 128 -
    // a larger grid starts later behind the kernel that produces the partials, a smaller one has longer load chains)
    const int rows = d->batch * d->num_q_heads;
    const Tune tune = desc_tune(d);
    int cluster = 1;
    if (p.total > 64 && !tune.off(HG_TUNE_NO_MERGE_CLUSTER)) cluster = rows <= 32 ? 8 : (rows <= 64 ? 4 : (rows <= 128 ? 2 : 1));
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)(rows * cluster));
    const bool big_cta = cluster == 1 && p.total > 256;            // many very long rows: 32 warps per row instead
    cfg.blockDim = dim3(big_cta ? 1024 : 256);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (!tune.off(HG_TUNE_NO_PDL)) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;     // start while the producer of the partials drains
        ++na;
    }
    if (cluster > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)cluster; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    auto launch = [&](auto k128, auto k64) { return d->head_dim == 128 ? cudaLaunchKernelEx(&cfg, k128, p) : cudaLaunchKernelEx(&cfg, k64, p); };
    cudaError_t e;
    // many rows: a warp per row, eight rows per CTA (a warp spends about 0.12 us per non-empty slot, a 1024-thread CTA
    // about 5 us per row whatever it finds: the warp wins from 2048 rows on, and from 1024 when rows are short)
    if ((rows >= 2048 || (rows >= 1024 && p.total <= 160)) && !tune.off(HG_TUNE_NO_MERGE_ROWS)) {
        cfg.gridDim = dim3((unsigned)((rows + 7) / 8));
        cfg.blockDim = dim3(256);
        e = d->head_dim == 128 ? cudaLaunchKernelEx(&cfg, merge_rows_kernel<128>, p, rows)
                               : cudaLaunchKernelEx(&cfg, merge_rows_kernel<64>, p, rows);
        if (e != cudaSuccess) { cudaGetLastError(); return HG_ERR_CUDA; }
        return HG_OK;
    }
    switch (cluster) {
        case 8: e = launch(merge_kernel<128, 256, 8>, merge_kernel<64, 256, 8>); break;
        case 4: e = launch(merge_kernel<128, 256, 4>, merge_kernel<64, 256, 4>); break;
        case 2: e = launch(merge_kernel<128, 256, 2>, merge_kernel<64, 256, 2>); break;
        default:
            e = big_cta ? launch(merge_kernel<128, 1024, 1>, merge_kernel<64, 1024, 1>)
                        : launch(merge_kernel<128, 256, 1>, merge_kernel<64, 256, 1>);
            break;
    }
    if (e != cudaSuccess) { cudaGetLastError(); return HG_ERR_CUDA; }
    return HG_OK;
}

// ---- workspace layout for the fused entry points ---------------------------------------------------------

// The address at which the current device can read or write a host buffer directly (pinned or registered
// host memory under unified addressing), or NULL when it cannot (pageable memory, device memory).
static void* device_alias(const void* host_ptr) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
}

static size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

struct Workspace {
    size_t o_part, m_part, l_part;           // chunk partials
    size_t sched;                            // work counter of the partial kernel
    size_t q, seq_lens, tok_begin, tok_end;  // staging (host form only)
    size_t host_part;                        // staged host partials, n_host_partials * (D + 2) floats per row + slack
    size_t out, lse;
    size_t total;
};

static Workspace plan_workspace(const hg_attn_desc* d, int n_host_partials, int n_host_src) {
    Workspace w;
    const size_t rows = (size_t)d->batch * d->num_q_heads;
    size_t off = 0;
    w.o_part = off; off += up256(rows * d->num_chunks * d->head_dim * sizeof(float));
    w.m_part = off; off += up256(rows * d->num_chunks * sizeof(float));
    w.l_part = off; off += up256(rows * d->num_chunks * sizeof(float));
    w.sched = off; off += 256;
    w.q = off; off += up256(rows * d->head_dim * 2);
    w.seq_lens = off; off += up256((size_t)d->batch * 4);
    w.tok_begin = off; off += up256((size_t)d->batch * 4);
    w.tok_end = off; off += up256((size_t)d->batch * 4);
    w.host_part = off; off += up256(rows * (size_t)n_host_partials * (d->head_dim + 2) * sizeof(float)) + (size_t)n_host_src * 3 * 256;
    w.out = off; off += up256(rows * d->head_dim * sizeof(float));
    w.lse = off; off += up256(rows * sizeof(float));
    w.total = off;
    return w;
}

}  // namespace hg

using namespace hg;

extern "C" {

hg_status hg_attn_partial(const void* q, const void* k_cache, const void* v_cache, const int32_t* seq_lens,
                          const int32_t* tok_begin, const int32_t* tok_end, float* o_part, float* m_part, float* l_part,
                          void* stream, const hg_attn_desc* desc) {
    return run_partial(MODE_MHA, q, k_cache, v_cache, seq_lens, tok_begin, tok_end, o_part, m_part, l_part, nullptr,
                       stream, desc);
}

hg_status hg_kv_read_probe(const void* k_cache, const void* v_cache, const int32_t* seq_lens, const int32_t* tok_begin,
                           const int32_t* tok_end, uint32_t* sink, void* stream, const hg_attn_desc* desc) {
    return run_partial(MODE_PROBE, nullptr, k_cache, v_cache, seq_lens, tok_begin, tok_end, nullptr, nullptr, nullptr,
                       sink, stream, desc);
}

hg_status hg_attn_merge(const hg_partial_src* partials, int32_t n_src, float* out, float* lse, void* stream,
                        const hg_attn_desc* desc) {
    return run_merge(partials, n_src, out, lse, stream, desc);
}

hg_status hg_attn_partial_from_logits(const float* logits, const void* v_rows, const int32_t* n_sel, float* o_part,
                                      float* m_part, float* l_part, void* stream, const hg_logits_desc* d) {
    if (!d || d->struct_size < offsetof(hg_logits_desc, status)) return HG_ERR_INVALID_ARG;
    if (d->batch < 1 || d->batch > 65535 || d->num_kv_heads < 1 || d->num_kv_heads > 65535 || d->num_q_heads < 1 ||
        d->num_q_heads % d->num_kv_heads)
        return HG_ERR_INVALID_ARG;
    if (d->head_dim <= 0 || d->head_dim % 8) return HG_ERR_INVALID_ARG;
    if (d->head_dim != 64 && d->head_dim != 128) return HG_ERR_UNSUPPORTED;
    if (d->dtype != HG_DTYPE_F16 && d->dtype != HG_DTYPE_BF16) return HG_ERR_INVALID_ARG;
    if (d->max_selected < 1 || d->chunk_tokens < 32 || d->chunk_tokens % 32 || d->num_chunks < 1) return HG_ERR_INVALID_ARG;
    if (d->chunk_tokens > LG_MAX_CHUNK) return HG_ERR_UNSUPPORTED;
    if ((int64_t)d->num_chunks * d->chunk_tokens < d->max_selected) return HG_ERR_INVALID_ARG;
    if ((int64_t)d->batch * d->num_kv_heads * d->max_selected > 0x7fffffffll) return HG_ERR_UNSUPPORTED;   // row coordinate
    if (!logits || !v_rows || !n_sel || !o_part || !m_part || !l_part) return HG_ERR_INVALID_ARG;
    if (!aligned16(v_rows) || !aligned16(o_part)) return HG_ERR_INVALID_ARG;
    LogitsParams p;
    memset(&p, 0, sizeof p);
    p.logits = logits; p.n_sel = n_sel; p.o_part = o_part; p.m_part = m_part; p.l_part = l_part;
    p.status = d->struct_size >= sizeof(hg_logits_desc) ? d->status : nullptr;
    p.B = d->batch; p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.G = p.Hq / p.Hkv; p.K = d->max_selected;
    p.chunk = d->chunk_tokens; p.NC = d->num_chunks;
    // the V rows as a 3-D tensor {component within a 64-element half, row, half}; one box is 64 rows of all halves,
    // 128-byte swizzled: the tile layout of hg_attn_partial
    EncodeTiledFn enc = encode_fn();
    if (!enc) return HG_ERR_CUDA;
    const int halves = d->head_dim / 64;
    CUtensorMap tv;
    cuuint64_t dims[3] = {64, (cuuint64_t)d->batch * d->num_kv_heads * d->max_selected, (cuuint64_t)halves};
    cuuint64_t strides[2] = {(cuuint64_t)d->head_dim * 2u, 128u};
    cuuint32_t box[3] = {64, (cuuint32_t)LG_TILE, (cuuint32_t)halves};
    cuuint32_t estr[3] = {1, 1, 1};
    if (enc(&tv, d->dtype == HG_DTYPE_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
            const_cast<void*>(v_rows), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return HG_ERR_UNSUPPORTED;
    dim3 grid((unsigned)p.NC, (unsigned)p.Hkv, (unsigned)p.B);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const bool bf16 = d->dtype == HG_DTYPE_BF16;
    auto launch = [&](auto kern, size_t smem) -> hg_status {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            cudaGetLastError();
            return HG_ERR_CUDA;
        }
        kern<<<grid, LG_THREADS, smem, cs>>>(tv, p);
        return cudaGetLastError() == cudaSuccess ? HG_OK : HG_ERR_CUDA;
    };
    const uint32_t ltune = d->struct_size >= offsetof(hg_logits_desc, tune) + sizeof(uint32_t) ? d->tune : 0u;
    const int tc_stages = d->head_dim == 128 ? lgtc_stages<128>(p.chunk) : lgtc_stages<64>(p.chunk);
    const long long tc_items = (long long)p.B * p.Hkv * p.NC * ((p.G + 7) / 8);
    // The library's choice: the tcgen05 kernel pays a hand-shake per work item and wins from 512-slot chunks on
    // (6-14 % at D = 128); with 256-slot chunks and at D = 64 the warp-level kernel, one CTA per chunk, is 7-10 % ahead.
    const bool tc_possible = tc_stages >= 2 && tc_items < 0x7fffffffll;
    const bool use_tc = tc_possible && !(ltune & HG_LOGITS_TUNE_WARP_MMA) &&
                        ((ltune & HG_LOGITS_TUNE_TCGEN05) != 0 || (d->head_dim == 128 && d->chunk_tokens >= 512));
    if (use_tc) {
        // the contraction on tcgen05.mma, the accumulator in tensor memory: persistent CTAs, two per SM
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
            cudaGetLastError();
            return HG_ERR_CUDA;
        }
        p.stages = tc_stages;
        p.head_blocks = (p.G + 7) / 8;
        p.items = (long long)p.B * p.Hkv * p.NC * p.head_blocks;
        const long long resident = (long long)LGTC_CTAS_PER_SM * sms;
        const unsigned ctas = (unsigned)(p.items < resident ? p.items : resident);
        auto launch_tc = [&](auto kern, size_t smem) -> hg_status {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
                cudaGetLastError();
                return HG_ERR_CUDA;
            }
            kern<<<ctas, LGTC_THREADS, smem, cs>>>(tv, p);
            return cudaGetLastError() == cudaSuccess ? HG_OK : HG_ERR_CUDA;
        };
        if (d->head_dim == 128)
            return bf16 ? launch_tc(logits_partial_tc_kernel<128, true>, logits_tc_smem_bytes<128>(p.chunk))
                        : launch_tc(logits_partial_tc_kernel<128, false>, logits_tc_smem_bytes<128>(p.chunk));
        return bf16 ? launch_tc(logits_partial_tc_kernel<64, true>, logits_tc_smem_bytes<64>(p.chunk))
                    : launch_tc(logits_partial_tc_kernel<64, false>, logits_tc_smem_bytes<64>(p.chunk));
    }
    if (d->head_dim == 128)
        return bf16 ? launch(logits_partial_kernel<128, true>, logits_smem_bytes<128>(p.chunk))
                    : launch(logits_partial_kernel<128, false>, logits_smem_bytes<128>(p.chunk));
    return bf16 ? launch(logits_partial_kernel<64, true>, logits_smem_bytes<64>(p.chunk))
                : launch(logits_partial_kernel<64, false>, logits_smem_bytes<64>(p.chunk));
}

int32_t hg_attn_suggest_chunk(int64_t total_tokens, int32_t num_q_heads, int32_t num_kv_heads, int32_t page_size) {
    if (total_tokens < 0 || num_kv_heads < 1 || num_q_heads < 1 || num_q_heads % num_kv_heads) return 0;
    const int shift = ilog2_exact(page_size);
    if (shift < 4 || shift > 8) return 0;
    const int G = num_q_heads / num_kv_heads;
    const int64_t rows = (int64_t)num_kv_heads * (G <= 8 ? 1 : (G + 15) / 16);     // items per chunk of one sequence
    // about fifteen items per resident CTA of a 148-SM device: items of 256-400 KB were the fastest at every size
    // measured (the last wave of work items ends spread over about one item's duration, so short items keep the tail
    // short; below that the per-item epilogues and the longer merge rows cost more than the tail gives back)
    const int64_t target_items = 4400;
    const int unit = page_size > TILE_T ? page_size : TILE_T;
    int64_t chunk = total_tokens * rows / target_items;
    chunk = (chunk + unit - 1) / unit * unit;
    const int64_t lo = 128 > unit ? 128 : unit, hi = 1024 > unit ? 1024 : unit;
    if (chunk < lo) chunk = lo;
    if (chunk > hi) chunk = hi;
    return (int32_t)chunk;
}

size_t hg_attn_workspace_bytes(const hg_attn_desc* desc, int32_t n_host_partials) {
    if (check_desc(desc, true) != HG_OK || n_host_partials < 0) return 0;
    return plan_workspace(desc, n_host_partials, HG_MAX_MERGE_SRC).total;
}

static hg_status decode_impl(const void* q, const void* k_cache, const void* v_cache, const int32_t* seq_lens,
                             const int32_t* tok_begin, const int32_t* tok_end, const hg_partial_src* host_partials,
                             int32_t n_host_src, float* out, float* lse, void* workspace, size_t workspace_bytes, void* stream,
                             const hg_attn_desc* desc, bool counter_is_zero) {
    hg_status st = check_desc(desc, true);
    if (st != HG_OK) return st;
    if (n_host_src < 0 || n_host_src > HG_MAX_MERGE_SRC - 1 || (n_host_src && !host_partials)) return HG_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HG_ERR_INVALID_ARG;
    const Workspace w = plan_workspace(desc, 0, 0);
    if (workspace_bytes < w.q) return HG_ERR_WORKSPACE;          // only the chunk partials are needed here
    char* ws = static_cast<char*>(workspace);
    float* o_part = reinterpret_cast<float*>(ws + w.o_part);
    float* m_part = reinterpret_cast<float*>(ws + w.m_part);
    float* l_part = reinterpret_cast<float*>(ws + w.l_part);
    hg_attn_desc dd;
    memset(&dd, 0, sizeof dd);
    memcpy(&dd, desc, desc->struct_size < sizeof dd ? desc->struct_size : sizeof dd);
    dd.struct_size = sizeof dd;
    dd.sched_counter = reinterpret_cast<int32_t*>(ws + w.sched);       // the workspace provides the work counter, and
    // HG_FLAG_COUNTER_CLEAN, if given, speaks about that one (a workspace zero-filled before its first use)
    dd.flags |= HG_FLAG_SPARSE_EMPTY;                                  // the chunk partials are private to this call and its merge
    st = run_partial(MODE_MHA, q, k_cache, v_cache, seq_lens, tok_begin, tok_end, o_part, m_part, l_part, nullptr, stream, &dd,
                     counter_is_zero);
    if (st != HG_OK) return st;
    hg_partial_src src[HG_MAX_MERGE_SRC];
    src[0].o = o_part; src[0].m = m_part; src[0].l = l_part; src[0].nc = desc->num_chunks; src[0].reserved = 0;
    for (int i = 0; i < n_host_src; ++i) src[1 + i] = host_partials[i];
    return run_merge(src, 1 + n_host_src, out, lse, stream, desc);
}

hg_status hg_attn_decode(const void* q, const void* k_cache, const void* v_cache, const int32_t* seq_lens,
                         const int32_t* tok_begin, const int32_t* tok_end, const hg_partial_src* host_partials,
                         int32_t n_host_src, float* out, float* lse, void* workspace, size_t workspace_bytes, void* stream,
                         const hg_attn_desc* desc) {
    return decode_impl(q, k_cache, v_cache, seq_lens, tok_begin, tok_end, host_partials, n_host_src, out, lse, workspace,
                       workspace_bytes, stream, desc, false);
}

hg_status hg_attn_decode_host(const void* q_host, const void* k_cache, const void* v_cache, const int32_t* seq_lens_host,
                              const int32_t* tok_begin_host, const int32_t* tok_end_host,
                              const hg_partial_src* host_partials_host, int32_t n_host_src, float* out_host, float* lse_host,
                              void* workspace, size_t workspace_bytes, void* stream, const hg_attn_desc* desc) {
    hg_status st = check_desc(desc, true);
    if (st != HG_OK) return st;
    if (!q_host || !seq_lens_host || !tok_begin_host || !tok_end_host || !out_host) return HG_ERR_INVALID_ARG;
    if (n_host_src < 0 || n_host_src > HG_MAX_MERGE_SRC - 1 || (n_host_src && !host_partials_host)) return HG_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HG_ERR_INVALID_ARG;
    int n_host_partials = 0;
    for (int i = 0; i < n_host_src; ++i) {
        const hg_partial_src& s = host_partials_host[i];
        if (!s.o || !s.m || !s.l || s.nc < 1) return HG_ERR_INVALID_ARG;
        n_host_partials += s.nc;
    }
    const Workspace w = plan_workspace(desc, n_host_partials, n_host_src);
    if (workspace_bytes < w.total) return HG_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const size_t rows = (size_t)desc->batch * desc->num_q_heads;
    const int D = desc->head_dim;
    // Fast path when the device can address every host buffer: one kernel stages q and the ranges, the merge
    // reads the host partials and writes the results in place - no copy-engine transfers at all.
    if (!desc_tune(desc).off(HG_TUNE_NO_HOST_DIRECT) && rows * D * 2 < (1ull << 32)) {
        StageParams sp;
        memset(&sp, 0, sizeof sp);
        const void* in[4] = {q_host, seq_lens_host, tok_begin_host, tok_end_host};
        const size_t at[4] = {w.q, w.seq_lens, w.tok_begin, w.tok_end};
        const size_t nb[4] = {rows * D * 2, (size_t)desc->batch * 4, (size_t)desc->batch * 4, (size_t)desc->batch * 4};
        bool direct = true;
        for (int i = 0; i < 4 && direct; ++i) {
            sp.src[i] = device_alias(in[i]); sp.dst[i] = ws + at[i]; sp.bytes[i] = (uint32_t)nb[i];
            direct = sp.src[i] != nullptr;
        }
        sp.n = 4;
        hg_partial_src alias[HG_MAX_MERGE_SRC];
        for (int i = 0; i < n_host_src && direct; ++i) {
            const hg_partial_src& s = host_partials_host[i];
            alias[i].nc = s.nc; alias[i].reserved = 0;
            alias[i].o = static_cast<const float*>(device_alias(s.o));
            alias[i].m = static_cast<const float*>(device_alias(s.m));
            alias[i].l = static_cast<const float*>(device_alias(s.l));
            direct = alias[i].o && alias[i].m && alias[i].l && aligned16(alias[i].o);
        }
        float* out_alias = direct ? static_cast<float*>(device_alias(out_host)) : nullptr;
        float* lse_alias = direct && lse_host ? static_cast<float*>(device_alias(lse_host)) : nullptr;
        direct = direct && out_alias && (!lse_host || lse_alias);
        if (direct) {
            sp.zero = reinterpret_cast<int32_t*>(ws + w.sched);        // the staging kernel also clears the work counter
            const unsigned blocks = (unsigned)((rows * D * 2 / 16 + STAGE_THREADS - 1) / STAGE_THREADS);
            stage_kernel<<<blocks < 1 ? 1 : (blocks > 64 ? 64 : blocks), STAGE_THREADS, 0, cs>>>(sp);
            if (cudaGetLastError() != cudaSuccess) return HG_ERR_CUDA;
            return decode_impl(ws + w.q, k_cache, v_cache, reinterpret_cast<const int32_t*>(ws + w.seq_lens),
                               reinterpret_cast<const int32_t*>(ws + w.tok_begin),
                               reinterpret_cast<const int32_t*>(ws + w.tok_end), alias, n_host_src, out_alias, lse_alias,
                               workspace, workspace_bytes, stream, desc, true);
        }
    }
    bool ok = true;
    ok &= cudaMemcpyAsync(ws + w.q, q_host, rows * D * 2, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    ok &= cudaMemcpyAsync(ws + w.seq_lens, seq_lens_host, (size_t)desc->batch * 4, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    ok &= cudaMemcpyAsync(ws + w.tok_begin, tok_begin_host, (size_t)desc->batch * 4, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    ok &= cudaMemcpyAsync(ws + w.tok_end, tok_end_host, (size_t)desc->batch * 4, cudaMemcpyHostToDevice, cs) == cudaSuccess;
    hg_partial_src dev_src[HG_MAX_MERGE_SRC];
    size_t off = w.host_part;
    for (int i = 0; i < n_host_src && ok; ++i) {
        const hg_partial_src& s = host_partials_host[i];
        const size_t ob = rows * s.nc * D * sizeof(float), mb = rows * s.nc * sizeof(float);
        dev_src[i].nc = s.nc; dev_src[i].reserved = 0;
        dev_src[i].o = reinterpret_cast<const float*>(ws + off);
        ok &= cudaMemcpyAsync(ws + off, s.o, ob, cudaMemcpyHostToDevice, cs) == cudaSuccess; off += up256(ob);
        dev_src[i].m = reinterpret_cast<const float*>(ws + off);
        ok &= cudaMemcpyAsync(ws + off, s.m, mb, cudaMemcpyHostToDevice, cs) == cudaSuccess; off += up256(mb);
        dev_src[i].l = reinterpret_cast<const float*>(ws + off);
        ok &= cudaMemcpyAsync(ws + off, s.l, mb, cudaMemcpyHostToDevice, cs) == cudaSuccess; off += up256(mb);
    }
    if (!ok) { cudaGetLastError(); return HG_ERR_CUDA; }
    float* out_dev = reinterpret_cast<float*>(ws + w.out);
    float* lse_dev = reinterpret_cast<float*>(ws + w.lse);
    st = hg_attn_decode(ws + w.q, k_cache, v_cache, reinterpret_cast<const int32_t*>(ws + w.seq_lens),
                        reinterpret_cast<const int32_t*>(ws + w.tok_begin), reinterpret_cast<const int32_t*>(ws + w.tok_end),
                        dev_src, n_host_src, out_dev, lse_dev, workspace, workspace_bytes, stream, desc);
    if (st != HG_OK) return st;
    ok &= cudaMemcpyAsync(out_host, out_dev, rows * D * sizeof(float), cudaMemcpyDeviceToHost, cs) == cudaSuccess;
    if (lse_host) ok &= cudaMemcpyAsync(lse_host, lse_dev, rows * sizeof(float), cudaMemcpyDeviceToHost, cs) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return HG_ERR_CUDA; }
    return HG_OK;
}

static KvPoolView pool_view(const hg_attn_desc* d, const void* k, const void* v) {
    KvPoolView pv;
    pv.k = static_cast<uint16_t*>(const_cast<void*>(k));
    pv.v = static_cast<uint16_t*>(const_cast<void*>(v));
    pv.block_table = d->block_table;
    pv.page_stride = d->page_stride; pv.head_stride = d->head_stride; pv.tok_stride = d->tok_stride;
    pv.B = d->batch; pv.Hkv = d->num_kv_heads; pv.D = d->head_dim; pv.page_size = d->page_size;
    pv.page_shift = ilog2_exact(d->page_size); pv.max_pages = d->max_pages; pv.num_pages = d->num_pages;
    return pv;
}

// The KV addressing fields only (chunking is irrelevant to residency operations).
static hg_status check_pool(const hg_attn_desc* d) {
    if (!d || d->struct_size < offsetof(hg_attn_desc, sched_counter)) return HG_ERR_INVALID_ARG;
    hg_attn_desc t;
    memset(&t, 0, sizeof t);
    memcpy(&t, d, d->struct_size < sizeof t ? d->struct_size : sizeof t);
    t.chunk_tokens = t.page_size > TILE_T ? t.page_size : TILE_T;
    t.num_chunks = 1;
    t.sched_counter = nullptr;
    t.struct_size = sizeof t;
    return check_desc(&t, true);
}

hg_status hg_kv_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache, int32_t* seq_lens,
                       int32_t* tok_end, void* stream, const hg_attn_desc* desc) {
    hg_status st = check_pool(desc);
    if (st != HG_OK) return st;
    if (!k_new || !v_new || !k_cache || !v_cache || !seq_lens) return HG_ERR_INVALID_ARG;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache)) return HG_ERR_INVALID_ARG;
    kv_append_kernel<<<desc->batch, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        pool_view(desc, k_cache, v_cache), static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new),
        seq_lens, tok_end, desc->status);
    return cudaGetLastError() == cudaSuccess ? HG_OK : HG_ERR_CUDA;
}

hg_status hg_kv_evict(const void* k_cache, const void* v_cache, int32_t* tok_begin, const int32_t* tok_end,
                      const int32_t* n_evict, int32_t max_evict, void* k_out, void* v_out, int32_t* freed_pages,
                      int32_t* n_freed, int32_t max_freed, void* stream, const hg_attn_desc* desc) {
    hg_status st = check_pool(desc);
    if (st != HG_OK) return st;
    if (!k_cache || !v_cache || !tok_begin || !tok_end || !n_evict || !k_out || !v_out) return HG_ERR_INVALID_ARG;
    if (max_evict < 1 || max_freed < 0 || (freed_pages && max_freed < 1)) return HG_ERR_INVALID_ARG;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_out) || !aligned16(v_out)) return HG_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const KvPoolView pv = pool_view(desc, k_cache, v_cache);
    dim3 grid((unsigned)((max_evict + EVICT_TOK_PER_CTA - 1) / EVICT_TOK_PER_CTA), (unsigned)desc->batch);
    kv_evict_copy_kernel<<<grid, 256, 0, cs>>>(pv, tok_begin, tok_end, n_evict, static_cast<uint16_t*>(k_out),
                                                static_cast<uint16_t*>(v_out), max_evict, desc->status);
    if (cudaGetLastError() != cudaSuccess) return HG_ERR_CUDA;
    kv_evict_commit_kernel<<<(desc->batch + 127) / 128, 128, 0, cs>>>(
        desc->batch, pv.page_shift, desc->max_pages, desc->num_pages, tok_begin, tok_end, n_evict, max_evict,
        const_cast<int32_t*>(desc->block_table), freed_pages, n_freed, max_freed);
    return cudaGetLastError() == cudaSuccess ? HG_OK : HG_ERR_CUDA;
}

hg_status hg_kv_evict_begin(int32_t* tok_begin, const int32_t* tok_end, const int32_t* n_evict, int32_t max_evict,
                            int32_t max_freed, int32_t* src_begin, int32_t* n_moved, void* stream, const hg_attn_desc* desc) {
    hg_status st = check_pool(desc);
    if (st != HG_OK) return st;
    if (!tok_begin || !tok_end || !n_evict || !src_begin || !n_moved || max_evict < 1 || max_freed < 0) return HG_ERR_INVALID_ARG;
    kv_evict_begin_kernel<<<(desc->batch + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        desc->batch, ilog2_exact(desc->page_size), desc->max_pages, desc->num_pages, tok_begin, tok_end, n_evict, max_evict,
        desc->block_table, max_freed > 0 ? 1 : 0, max_freed, src_begin, n_moved, desc->status);
    return cudaGetLastError() == cudaSuccess ? HG_OK : HG_ERR_CUDA;
}

hg_status hg_kv_evict_copy(const void* k_cache, const void* v_cache, const int32_t* src_begin, const int32_t* n_moved,
                           int32_t max_evict, void* k_out, void* v_out, void* stream, const hg_attn_desc* desc) {
    hg_status st = check_pool(desc);
    if (st != HG_OK) return st;
    if (!k_cache || !v_cache || !src_begin || !n_moved || !k_out || !v_out || max_evict < 1) return HG_ERR_INVALID_ARG;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_out) || !aligned16(v_out)) return HG_ERR_INVALID_ARG;
    const KvPoolView pv = pool_view(desc, k_cache, v_cache);
    dim3 grid((unsigned)((max_evict + EVICT_TOK_PER_CTA - 1) / EVICT_TOK_PER_CTA), (unsigned)desc->batch);
    kv_evict_copy_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(pv, src_begin, nullptr, n_moved,
                                                                               static_cast<uint16_t*>(k_out),
                                                                               static_cast<uint16_t*>(v_out), max_evict, desc->status);
    return cudaGetLastError() == cudaSuccess ? HG_OK : HG_ERR_CUDA;
}

hg_status hg_kv_evict_finish(const int32_t* src_begin, const int32_t* n_moved, int32_t* freed_pages, int32_t* n_freed,
                             int32_t max_freed, void* stream, const hg_attn_desc* desc) {
    hg_status st = check_pool(desc);
    if (st != HG_OK) return st;
    if (!src_begin || !n_moved || max_freed < 0 || (freed_pages && max_freed < 1)) return HG_ERR_INVALID_ARG;
    kv_evict_finish_kernel<<<(desc->batch + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        desc->batch, ilog2_exact(desc->page_size), desc->max_pages, src_begin, n_moved, const_cast<int32_t*>(desc->block_table),
        freed_pages, n_freed, max_freed);
    return cudaGetLastError() == cudaSuccess ? HG_OK : HG_ERR_CUDA;
}

const char* hg_status_string(hg_status s) {
    switch (s) {
        case HG_OK: return "ok";
        case HG_ERR_INVALID_ARG: return "invalid argument";
        case HG_ERR_UNSUPPORTED: return "unsupported configuration";
        case HG_ERR_CUDA: return "CUDA error";
        case HG_ERR_WORKSPACE: return "workspace too small";
        default: return "unknown status";
    }
}

uint32_t hg_version(void) { return HG_VERSION; }

}  // extern "C"

// ---- decode without any allocation: chunk partials in a fixed array of the device image ----------------

// Scratch for hg_attn_decode_static.  In host code this name is only a handle for the symbol, not a
// device address: the address is obtained once per device with cudaGetSymbolAddress.
// (the 256 bytes behind the partials hold the partial kernel's work counter)
static __device__ __align__(256) unsigned char hg_static_scratch[HG_STATIC_SCRATCH_BYTES + 256];

static std::atomic<void*> g_static_scratch_addr[hg::kMaxDevices];

// Device address of the scratch array on the current device (looked up on the first call per device).
static void* static_scratch_ptr() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= hg::kMaxDevices) { cudaGetLastError(); return nullptr; }
    void* p = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (p) return p;
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, hg_static_scratch) != cudaSuccess || !addr) { cudaGetLastError(); return nullptr; }
    g_static_scratch_addr[dev].store(addr, std::memory_order_release);   // every thread would store the same value
    return addr;
}

extern "C" hg_status hg_attn_decode_static(const void* q, const void* k_cache, const void* v_cache,
                                           const int32_t* seq_lens, const int32_t* tok_begin, const int32_t* tok_end,
                                           const hg_partial_src* host_partials, int32_t n_host_src, float* out,
                                           float* lse, void* stream, const hg_attn_desc* desc) {
    hg_status st = hg::check_desc(desc, true);
    if (st != HG_OK) return st;
    const hg::Workspace w = hg::plan_workspace(desc, 0, 0);
    if (w.sched > HG_STATIC_SCRATCH_BYTES) return HG_ERR_WORKSPACE;     // the three partial arrays exceed the fixed scratch
    void* scratch = static_scratch_ptr();
    if (!scratch) return HG_ERR_CUDA;
    return hg_attn_decode(q, k_cache, v_cache, seq_lens, tok_begin, tok_end, host_partials, n_host_src, out, lse,
                          scratch, HG_STATIC_SCRATCH_BYTES + 256, stream, desc);
}
