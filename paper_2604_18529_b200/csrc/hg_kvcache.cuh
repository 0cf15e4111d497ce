// KV residency operations on the paged pool (sm_100a): appending the current step's K/V rows and
// moving the oldest tokens of the GPU slice out (the eviction engine's device half).  Pure data
// movement: 16-byte vector copies, no arithmetic.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace hg {

struct KvPoolView {
    uint16_t* k;
    uint16_t* v;
    const int32_t* block_table;   // may be NULL: identity paging
    int64_t page_stride, head_stride, tok_stride;
    int B, Hkv, D, page_size, page_shift, max_pages, num_pages;
};

// Physical page of token t of sequence b, or -1 if it is not resident / out of range.
__device__ __forceinline__ int kv_page_of(const KvPoolView& pv, int b, int t) {
    const int pg = t >> pv.page_shift;
    if (t < 0 || pg >= pv.max_pages) return -1;
    const int phys = pv.block_table ? pv.block_table[(size_t)b * pv.max_pages + pg] : b * pv.max_pages + pg;
    return (phys < 0 || phys >= pv.num_pages) ? -1 : phys;
}

// One CTA per sequence: rows k_new / v_new [B][Hkv][D] go to position seq_lens[b]; then seq_lens[b]
// (and tok_end[b], if given and equal to the old length) grow by one.
__global__ void kv_append_kernel(KvPoolView pv, const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                                 int32_t* seq_lens, int32_t* tok_end, int32_t* status) {
    const int b = blockIdx.x;
    const int t = seq_lens[b];
    const int old_end = tok_end ? tok_end[b] : 0;
    const int phys = kv_page_of(pv, b, t);
    __syncthreads();                                   // everybody has read the old length
    if (phys < 0) {
        if (threadIdx.x == 0 && status) atomicOr(status, HG_DEV_BAD_PAGE);
        return;
    }
    const int vec_per_row = pv.D / 8;                  // 16-byte vectors
    const int64_t base = (int64_t)phys * pv.page_stride + (int64_t)(t & (pv.page_size - 1)) * pv.tok_stride;
    for (int i = threadIdx.x; i < pv.Hkv * vec_per_row; i += blockDim.x) {
        const int g = i / vec_per_row, c = i - g * vec_per_row;
        const int64_t dst = base + (int64_t)g * pv.head_stride + c * 8;
        const int64_t src = ((int64_t)b * pv.Hkv + g) * pv.D + c * 8;
        *reinterpret_cast<uint4*>(pv.k + dst) = *reinterpret_cast<const uint4*>(k_new + src);
        *reinterpret_cast<uint4*>(pv.v + dst) = *reinterpret_cast<const uint4*>(v_new + src);
    }
    if (threadIdx.x == 0) {
        seq_lens[b] = t + 1;
        if (tok_end && old_end == t) tok_end[b] = t + 1;
    }
}

constexpr int EVICT_TOK_PER_CTA = 8;

// Copies the first n_evict[b] tokens of the slice [tok_begin, tok_end) of every sequence into
// k_out / v_out [B][max_evict][Hkv][D] (token-major rows, the layout the host keeps its part in).
// Grid (token blocks, B); reads only.
__global__ void kv_evict_copy_kernel(KvPoolView pv, const int32_t* __restrict__ tok_begin, const int32_t* __restrict__ tok_end,
                                     const int32_t* __restrict__ n_evict, uint16_t* k_out, uint16_t* v_out, int max_evict,
                                     int32_t* status) {
    const int b = blockIdx.y;
    const int tb = tok_begin[b];
    // (three-step form: tok_begin / n_evict are the recorded range, tok_end is absent)
    const int ne = max(0, min(min(n_evict[b], max_evict), tok_end ? tok_end[b] - tb : max_evict));
    const int vec_per_row = pv.D / 8, vec_per_tok = pv.Hkv * vec_per_row;
    const int i0 = blockIdx.x * EVICT_TOK_PER_CTA, i1 = min(ne, i0 + EVICT_TOK_PER_CTA);
    __shared__ int s_phys[EVICT_TOK_PER_CTA];          // one block-table look-up per token, not per vector
    if ((int)threadIdx.x < i1 - i0) {
        const int phys = kv_page_of(pv, b, tb + i0 + threadIdx.x);
        s_phys[threadIdx.x] = phys;
        if (phys < 0 && status) atomicOr(status, HG_DEV_BAD_PAGE);
    }
    __syncthreads();
    const int n_vec = (i1 - i0) * vec_per_tok;
    constexpr int UNROLL = 4;                           // independent 16-byte K and V loads in flight per thread
    for (int base = threadIdx.x; base < n_vec; base += UNROLL * blockDim.x) {
        uint4 kk[UNROLL], vv[UNROLL];
        int64_t dst[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int idx = base + u * blockDim.x;
            dst[u] = -1;
            if (idx >= n_vec) continue;
            const int i = idx / vec_per_tok, r = idx - i * vec_per_tok;
            const int g = r / vec_per_row, c = r - g * vec_per_row;
            const int phys = s_phys[i];
            if (phys < 0) continue;
            const int t = tb + i0 + i;
            const int64_t src = (int64_t)phys * pv.page_stride + (int64_t)(t & (pv.page_size - 1)) * pv.tok_stride +
                                (int64_t)g * pv.head_stride + c * 8;
            dst[u] = (((int64_t)b * max_evict + i0 + i) * pv.Hkv + g) * pv.D + c * 8;
            kk[u] = *reinterpret_cast<const uint4*>(pv.k + src);
            vv[u] = *reinterpret_cast<const uint4*>(pv.v + src);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            if (dst[u] < 0) continue;
            *reinterpret_cast<uint4*>(k_out + dst[u]) = kk[u];
            *reinterpret_cast<uint4*>(v_out + dst[u]) = vv[u];
        }
    }
}

// Which rows leave sequence b: [tb, nb).  ne = min(n_evict, max_evict, slice length) rows are asked for; the range is
// cut back to nothing when it meets an unmapped or out-of-pool block-table entry (no token may be lost from both
// tiers), and, when the emptied pages are to be listed, to the first page that does not fit a list of max_freed
// entries (no page is un-mapped whose id cannot be reported).
struct EvictRange { int tb, nb; };

__device__ __forceinline__ EvictRange evict_range(int b, int page_shift, int max_pages, int num_pages, const int32_t* tok_begin,
                                                  const int32_t* tok_end, const int32_t* n_evict, int max_evict,
                                                  const int32_t* block_table, bool listed, int max_freed) {
    EvictRange r;
    r.tb = tok_begin[b];
    const int ne = max(0, min(min(n_evict[b], max_evict), tok_end[b] - r.tb));
    r.nb = r.tb + ne;
    if (!block_table || ne == 0) return r;
    const int first_pg = r.tb >> page_shift;
    for (int pg = first_pg; pg <= ((r.nb - 1) >> page_shift); ++pg) {
        const int phys = pg < max_pages ? block_table[(size_t)b * max_pages + pg] : -1;
        if (phys < 0 || phys >= num_pages) { r.nb = r.tb; return r; }
    }
    // pages wholly below the new beginning leave; a partly used page stays mapped (it may still take appended rows)
    if (listed && (r.nb >> page_shift) - first_pg > max_freed) r.nb = (first_pg + max_freed) << page_shift;
    return r;
}

// Un-maps the pages wholly below nb (starting at tb's page) and lists them.  One thread's work for one sequence.
__device__ __forceinline__ void evict_unmap(int b, int page_shift, int max_pages, EvictRange r, int32_t* block_table,
                                            int32_t* freed, int32_t* n_freed, int max_freed) {
    int cnt = 0;
    if (block_table)
        for (int pg = r.tb >> page_shift; pg < (r.nb >> page_shift) && pg < max_pages; ++pg) {
            if (freed && cnt < max_freed) freed[(size_t)b * max_freed + cnt] = block_table[(size_t)b * max_pages + pg];
            ++cnt;
            block_table[(size_t)b * max_pages + pg] = -1;
        }
    if (freed) for (int i = cnt; i < max_freed; ++i) freed[(size_t)b * max_freed + i] = -1;
    if (n_freed) n_freed[b] = cnt;
}

// After the copy (one-call form): advances tok_begin, un-maps the pages that no longer hold a token of the slice and
// lists their physical ids in freed [B][max_freed] (-1 padded), n_freed [B].  One thread per sequence.
__global__ void kv_evict_commit_kernel(int B, int page_shift, int max_pages, int num_pages, int32_t* tok_begin,
                                       const int32_t* tok_end, const int32_t* n_evict, int max_evict, int32_t* block_table,
                                       int32_t* freed, int32_t* n_freed, int max_freed) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const EvictRange r = evict_range(b, page_shift, max_pages, num_pages, tok_begin, tok_end, n_evict, max_evict, block_table,
                                     freed != nullptr, max_freed);
    evict_unmap(b, page_shift, max_pages, r, block_table, freed, n_freed, max_freed);
    tok_begin[b] = r.nb;
}

// Three-step form, for an eviction that drains beside the attention of the same step.
// Step 1 (on the attention's stream, before it): decides the range, records it in src_begin / n_moved and moves
// tok_begin, so that whatever follows on this stream already works on the shrunk slice.  The block table is left
// alone: the rows are still where the table says.
__global__ void kv_evict_begin_kernel(int B, int page_shift, int max_pages, int num_pages, int32_t* tok_begin,
                                      const int32_t* tok_end, const int32_t* n_evict, int max_evict,
                                      const int32_t* block_table, int listed, int max_freed, int32_t* src_begin,
                                      int32_t* n_moved, int32_t* status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const EvictRange r = evict_range(b, page_shift, max_pages, num_pages, tok_begin, tok_end, n_evict, max_evict, block_table,
                                     listed != 0, max_freed);
    const int asked = max(0, min(min(n_evict[b], max_evict), tok_end[b] - r.tb));
    if (r.nb == r.tb && asked > 0 && status) atomicOr(status, HG_DEV_BAD_PAGE);
    src_begin[b] = r.tb;
    n_moved[b] = r.nb - r.tb;
    tok_begin[b] = r.nb;
}

// Step 3 (any stream, after step 2's copy kernel): un-maps and lists the pages below the new beginning.  These
// block-table entries belong to pages no attention over the shrunk slice looks up.
__global__ void kv_evict_finish_kernel(int B, int page_shift, int max_pages, const int32_t* src_begin, const int32_t* n_moved,
                                       int32_t* block_table, int32_t* freed, int32_t* n_freed, int max_freed) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    EvictRange r;
    r.tb = src_begin[b];
    r.nb = r.tb + n_moved[b];
    evict_unmap(b, page_shift, max_pages, r, block_table, freed, n_freed, max_freed);
}

}  // namespace hg
