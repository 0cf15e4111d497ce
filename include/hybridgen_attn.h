/*
 * hybridgen_attn.h - C ABI of the B200 (sm_100a) decode-attention library for CPU-GPU hybrid
 * attention with the KV cache split along the token axis ("attention logit parallelism",
 * Section 4.2 of the HybridGen paper).
 *
 * The GPU holds a slice [tok_begin, tok_end) of every sequence's KV cache; the host holds the
 * rest.  Attention logits are independent per token (Section 4.2), so each side can process its
 * own tokens.  This library does the device side in two calls:
 *
 *   hg_attn_partial  per (sequence, query head, KV chunk): the scaled logits
 *                    s_t = <q, K_t> / sqrt(D) (Section 2.1), the chunk maximum m, the exp-sum
 *                    l = sum e^{s_t - m} and the un-normalised value aggregate
 *                    o = sum e^{s_t - m} V_t  (workflow step 4 plus the device-local part of step 5)
 *   hg_attn_merge    log-sum-exp combination of any number of such partials (GPU chunks and
 *                    partials for the host-held slice) into softmax(q K^T / sqrt(D)) V and its
 *                    log-sum-exp.  It stands for the Token Concatenator + softmax + value
 *                    aggregation of Section 4.2 / workflow step 5 and gives the same result as
 *                    monolithic attention over the union of the token sets.
 *
 * Conventions
 *   - Plain C linkage; all structs are PODs that start with their own size.
 *   - "dev" pointers are device memory, "host" pointers ordinary host memory.  The caller owns
 *     every buffer; except where an entry point says otherwise the library allocates nothing,
 *     keeps no mutable global state, never synchronises the device and never aborts.
 *   - Work is enqueued on the given CUDA stream (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) and runs asynchronously.
 *   - Every entry point returns an hg_status.  When validation fails nothing is launched.
 *   - m and lse are in natural-log units.  An empty chunk is (m, l, o) = (-inf, 0, 0); merging only
 *     empty sources gives out = 0, lse = -inf.  No NaN is produced for finite inputs.
 *   - Query head h reads KV head h / (num_q_heads / num_kv_heads) (consecutive grouping).
 *   - Decode step: the single query of a sequence attends every cached token of its slice; there
 *     is no mask inside the step (the new token's K, V are appended before attention, Section 2.1).
 */
#ifndef HYBRIDGEN_ATTN_H_
#define HYBRIDGEN_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HG_VERSION 0x00010000u /* major.minor.patch = 0.1.0 */

typedef enum hg_status {
    HG_OK = 0,
    HG_ERR_INVALID_ARG = 1, /* null pointer, bad size, misaligned base or stride, struct too small */
    HG_ERR_UNSUPPORTED = 2, /* valid but not implemented (head_dim, page size, group size ...) */
    HG_ERR_CUDA = 3,        /* a CUDA call or the launch failed (see cudaGetLastError) */
    HG_ERR_WORKSPACE = 4    /* caller workspace too small / problem exceeds a fixed scratch limit */
} hg_status;

typedef enum hg_dtype { HG_DTYPE_F16 = 0, HG_DTYPE_BF16 = 1 } hg_dtype;

/* bits of hg_attn_desc.flags */
#define HG_FLAG_NONE 0u
#define HG_FLAG_TEST_STALL 1u /* testing aid: the loader of hg_attn_partial / hg_kv_read_probe never fills a
                                 stage, so every wait runs into its time limit (about 2 s); the call then
                                 reports HG_DEV_WAIT_TIMEOUT through *status and returns normally */

#define HG_FLAG_SPARSE_EMPTY 2u /* empty chunk slots get m = -inf and l = 0 only; their o rows are left as they
                                   are (hg_attn_merge never reads the o of an empty partial).  For batches that
                                   mix long and short sequences: num_chunks is set by the longest one, and
                                   zero-filling every short sequence's unused slots can cost more than the
                                   attention itself.  hg_attn_decode and its variants always work this way on
                                   their own workspace. */

#define HG_FLAG_COUNTER_CLEAN 4u /* both words of sched_counter are zero when the call's kernel starts (for instance
                                   because the last thing that used them was an earlier call of this library that
                                   ended normally: every call leaves them at zero).  The call then enqueues no
                                   clearing in front of its kernel, which lets the kernel start as a programmatic
                                   dependent of whatever precedes it in the stream.  After a call that reported
                                   HG_DEV_WAIT_TIMEOUT clear the words yourself before using the flag again.
                                   hg_attn_decode and hg_attn_decode_static keep their work counter in the workspace
                                   (the static scratch): there the flag speaks about that counter - pass it only for a
                                   workspace that was zero-filled before its first use and has been used by this
                                   library alone since.  hg_attn_decode_host clears the counter on its way in any
                                   case. */

/* bits the kernels may set in *hg_attn_desc.status (device word, optional; several may be set at once) */
#define HG_DEV_OK 0
#define HG_DEV_WAIT_TIMEOUT 1 /* a bounded on-chip barrier wait ran out; the call's results are invalid.
                                 While this bit is set the kernels skip their work, so clear the word
                                 before the next call. */
#define HG_DEV_BAD_PAGE 2     /* a block-table entry of a resident page was outside [0, num_pages): the page was not
                                 read and its tokens were left out of the partial, as if they were not resident */
#define HG_DEV_RANGE 4        /* a slice reached past max_pages * page_size tokens, the end of its block-table row:
                                 it was cut there (the partials cover [tok_begin, max_pages * page_size)) */

/*
 * Problem description (host struct).
 *
 * KV pool addressing, in elements of the 16-bit dtype, for token t of sequence b, KV head g,
 * component d (the innermost D elements are contiguous):
 *     page   = block_table ? block_table[b * max_pages + t / page_size] : b * max_pages + t / page_size
 *     offset = page * page_stride + g * head_stride + (t % page_size) * tok_stride + d
 * K and V pools share this addressing.  Only pages that overlap [tok_begin, tok_end) are
 * dereferenced; other block-table entries may be -1.  Whole resident pages may be read,
 * including rows outside the slice, but such rows never influence a result.
 * "Token t" is a position in the block-table row, nothing more: a row that lists only chosen pages of a
 * sequence, in token order, with seq_lens / tok_end counted in that row's positions, gives attention over
 * exactly those pages (a page-granular token selection, Section 4.5, needs no other entry point).
 * Requirements: head_dim in {64, 128}; page_size in {16, 32, 64, 128, 256}; pool base addresses
 * 16-byte aligned; every stride a multiple of 8 elements; chunk_tokens a multiple of 64 and of
 * page_size, at most 512 pages.
 *
 * Chunk grid: chunks sit on absolute multiples of chunk_tokens.  Chunk c of sequence b covers
 *     [(tok_begin[b] / chunk_tokens + c) * chunk_tokens, + chunk_tokens)  intersected with
 *     [tok_begin[b], tok_end[b]),
 * so nc_b = ceil(tok_end / chunk_tokens) - floor(tok_begin / chunk_tokens) chunks are non-empty
 * (0 when the slice is empty).  num_chunks must be >= every nc_b; slots c >= nc_b are written as
 * empty partials.
 */
typedef struct hg_attn_desc {
    uint32_t struct_size;      /* sizeof(hg_attn_desc) as compiled by the caller */
    int32_t batch;             /* B  >= 1 */
    int32_t num_q_heads;       /* Hq, a multiple of num_kv_heads */
    int32_t num_kv_heads;      /* Hkv */
    int32_t head_dim;          /* D */
    int32_t dtype;             /* hg_dtype of q, K and V */
    int32_t page_size;         /* tokens per page */
    int32_t num_pages;         /* pages in each pool */
    int64_t page_stride;       /* elements */
    int64_t head_stride;       /* elements */
    int64_t tok_stride;        /* elements */
    const int32_t* block_table; /* dev [B][max_pages], or NULL for identity paging */
    int32_t max_pages;         /* row length of block_table */
    int32_t chunk_tokens;      /* C */
    int32_t num_chunks;        /* NC: chunk slots per (sequence, head) in o/m/l_part */
    float scale;               /* logit scale; 0 means 1/sqrt(D) */
    uint32_t flags;            /* HG_FLAG_* */
    int32_t* status;           /* dev, optional: receives HG_DEV_* if a kernel detects a problem */
    int32_t* sched_counter;    /* dev, optional, 8 bytes (two int32, 8-byte aligned): when given, the CTAs of
                                  hg_attn_partial draw work items from it dynamically (better balance on ragged
                                  batches); NULL: items are dealt round-robin.  The call clears both words on the
                                  stream in front of its kernel unless HG_FLAG_COUNTER_CLEAN says they are zero
                                  already; the kernel leaves them at zero when it ends normally.  Left alone when
                                  the problem has no more items than the device has resident CTAs.  Must not be
                                  shared by calls that may overlap on the GPU.  Present when struct_size covers it. */
    uint32_t tune;             /* HG_TUNE_* bits; 0 = the library's defaults.  Each bit switches one choice of the
                                  schedule off; results do not depend on them (the tests show equal bits), speed
                                  does.  Present when struct_size covers it, like the two fields below. */
    int32_t tune_stages;       /* depth of the shared-memory ring of hg_attn_partial, 2..8; 0 = default (3) */
    int32_t tune_ctas_per_sm;  /* upper limit on resident CTAs per SM for hg_attn_partial; 0 = as many as fit */
} hg_attn_desc;

/* bits of hg_attn_desc.tune */
#define HG_TUNE_NO_PERSISTENT 1u     /* one CTA per work item instead of a persistent grid */
#define HG_TUNE_NO_DYNAMIC 2u        /* deal items round-robin even when a work counter is given */
#define HG_TUNE_NO_PDL 4u            /* no programmatic dependent launches */
#define HG_TUNE_NO_MERGE_CLUSTER 8u  /* hg_attn_merge: never split a row over a thread-block cluster */
#define HG_TUNE_NO_MERGE_ROWS 16u    /* hg_attn_merge: never use the warp-per-row kernel */
#define HG_TUNE_NO_GQA16 32u         /* groups of more than 8 query heads as items of 8 heads, not 16 */
#define HG_TUNE_NO_HOST_DIRECT 64u   /* hg_attn_decode_host: always stage through the workspace with copies */
#define HG_TUNE_NO_SPEC_PREFETCH 128u /* a partial kernel launched as a programmatic dependent does not request its
                                        guessed first tiles into the L2 while it waits for its predecessor */

/* One source of partials for hg_attn_merge (host struct, dev pointers). */
typedef struct hg_partial_src {
    const float* o; /* dev [B][Hq][nc][D] */
    const float* m; /* dev [B][Hq][nc]    */
    const float* l; /* dev [B][Hq][nc]    */
    int32_t nc;     /* partials per (sequence, head) in this source, >= 1 */
    int32_t reserved;
} hg_partial_src;

/*
 * Scaled logits, chunk max, exp-sum and un-normalised P.V for the GPU-resident slice
 * (Section 2.1 for the logit definition; Section 4.2 and workflow step 4 for the token split).
 *
 *   q          dev [B][Hq][D], dtype as desc->dtype, 16-byte aligned
 *   k_cache    dev K pool, v_cache dev V pool (addressing above)
 *   seq_lens   dev int32 [B]   cached tokens per sequence
 *   tok_begin  dev int32 [B]   0 <= tok_begin <= tok_end <= seq_len; values outside are clipped to [0, seq_len]
 *   tok_end    dev int32 [B]
 *   o_part     dev float [B][Hq][NC][D]  out: sum_t e^{s_t - m} V_t
 *   m_part     dev float [B][Hq][NC]     out: exact fp32 chunk maximum of the scaled logits
 *   l_part     dev float [B][Hq][NC]     out: sum_t e^{s_t - m}
 * Ranges are read on the device, so the call never waits for the GPU; a slice that needs more
 * than num_chunks chunks is truncated to its first num_chunks chunks.
 * Accumulation is fp32.  For num_q_heads > num_kv_heads the P.V product runs on tensor cores with
 * P carried as a two-term (hi + lo) 16-bit expansion.
 * Errors: HG_ERR_INVALID_ARG / HG_ERR_UNSUPPORTED before any launch; HG_ERR_CUDA if the launch fails.
 */
hg_status hg_attn_partial(const void* q, const void* k_cache, const void* v_cache, const int32_t* seq_lens,
                          const int32_t* tok_begin, const int32_t* tok_end, float* o_part, float* m_part,
                          float* l_part, void* stream, const hg_attn_desc* desc);

/*
 * Log-sum-exp merge and normalisation (stands for concatenation + softmax + value aggregation of
 * Section 4.2 / workflow step 5; result identical, up to rounding order, to attention over the
 * union of the sources' token sets).
 *
 *   partials  host array of n_src sources (n_src >= 1); each source's arrays are dev memory
 *   out       dev float [B][Hq][D]   sum_i w_i o_i / sum_i w_i l_i,  w_i = e^{m_i - max_j m_j}
 *   lse       dev float [B][Hq]      max_j m_j + ln sum_i w_i l_i   (may be NULL)
 * A partial with m = -inf is empty: it contributes nothing and its o row is never read.
 * Only batch, num_q_heads and head_dim of desc are used.  n_src <= HG_MAX_MERGE_SRC.
 */
#define HG_MAX_MERGE_SRC 8
hg_status hg_attn_merge(const hg_partial_src* partials, int32_t n_src, float* out, float* lse, void* stream,
                        const hg_attn_desc* desc);

/*
 * A chunk size for a problem of `total_tokens` GPU-resident token positions (summed over the
 * sequences; an estimate will do) with the given head counts and page size: a multiple of 64 and of
 * page_size between 128 and 1024 tokens that gives every resident CTA of the device about fifteen
 * work items.  Chunk size is the caller's choice (the paper has no chunks); this is the rule the
 * measured workloads of this library follow: work items of 256-400 KB of K and V ran fastest at every
 * size (the last items of a launch end spread over one item's duration), small problems need short
 * chunks to spread over the SMs.  Returns 0 for invalid arguments.  No CUDA call is made.
 */
int32_t hg_attn_suggest_chunk(int64_t total_tokens, int32_t num_q_heads, int32_t num_kv_heads, int32_t page_size);

/*
 * Bytes of device workspace hg_attn_decode / hg_attn_decode_host need for this problem
 * (chunk partials, plus staging for q, ranges, host partials and results in the _host form).
 * n_host_partials is the total number of partials per (sequence, head) that the host sources of
 * hg_attn_decode_host will carry: the sum of their nc fields (a source of nc = 3 counts 3), not the
 * number of sources.  hg_attn_decode ignores it (its host partials are already on the device).
 * Returns 0 for an invalid description.
 */
size_t hg_attn_workspace_bytes(const hg_attn_desc* desc, int32_t n_host_partials);

/*
 * One pass of the whole path: hg_attn_partial into workspace, then hg_attn_merge of those
 * chunk partials with n_host_src further sources (partials for the host-held slice, already in
 * device memory).  workspace: dev, 256-byte aligned, at least hg_attn_workspace_bytes().
 */
hg_status hg_attn_decode(const void* q, const void* k_cache, const void* v_cache, const int32_t* seq_lens,
                         const int32_t* tok_begin, const int32_t* tok_end, const hg_partial_src* host_partials,
                         int32_t n_host_src, float* out, float* lse, void* workspace, size_t workspace_bytes,
                         void* stream, const hg_attn_desc* desc);

/*
 * The same pass for a caller whose per-step data lives in HOST memory: q, the three range arrays,
 * the host-slice partials (hg_partial_src with HOST pointers here) and the results out / lse are
 * host buffers.  When every one of them is pinned (or registered) host memory that the device can
 * address, no copy is enqueued at all: one small kernel stages q and the ranges into the
 * workspace, the merge reads the host partials and writes out / lse in place over the bus (the
 * host partial's o must then be 16-byte aligned).  Otherwise - pageable memory, or any buffer the
 * device cannot address - everything is staged through the device workspace with
 * cudaMemcpyAsync on the stream.  Either way the buffers are read and written when the stream
 * reaches the work, not at call time: leave them alone until the stream has been synchronised,
 * after which out / lse are valid.  The KV pools and the block table stay device resident - they
 * are the GPU's slice of the cache, not per-step input.  Returns after enqueuing.
 */
hg_status hg_attn_decode_host(const void* q_host, const void* k_cache, const void* v_cache,
                              const int32_t* seq_lens_host, const int32_t* tok_begin_host,
                              const int32_t* tok_end_host, const hg_partial_src* host_partials_host,
                              int32_t n_host_src, float* out_host, float* lse_host, void* workspace,
                              size_t workspace_bytes, void* stream, const hg_attn_desc* desc);

/*
 * hg_attn_decode for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry point exists for the embedding environment, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plugin whose host gives it a
 * fixed memory budget and forbids further allocation, a latency-critical decode loop that must
 * not take the allocator's lock or trigger the implicit device synchronisation cudaFree brings,
 * a component that is handed buffers by its framework and has no allocator of its own.  Such a
 * caller has the inputs and the output buffers but nowhere to put the chunk partials that sit
 * between the two kernels.
 *
 * Here those partials live in a fixed array inside the library's device image
 * (HG_STATIC_SCRATCH_BYTES bytes, reserved on every GPU that loads the library for as long as the
 * process lives).  Arguments and results are those of hg_attn_decode minus the workspace.
 *
 *   - Limit: with n = batch * num_q_heads * num_chunks, the three partial arrays - n * head_dim * 4
 *     bytes of o and twice n * 4 bytes of m and l, each array rounded up to a multiple of 256 bytes -
 *     must fit in HG_STATIC_SCRATCH_BYTES (exactly filling it is accepted); a larger problem is
 *     refused with HG_ERR_WORKSPACE and nothing is launched.  Use bigger chunks or hg_attn_decode
 *     instead.
 *   - The first call on each device looks up the array's device address (a symbol query, no
 *     allocation) with that device current.  Make that first call outside any stream capture.
 *   - Neither this call nor anything it calls uses cudaMalloc, cudaFree or an allocating library.
 *   - All calls on a device share the one array and it keeps the previous call's contents.  Every
 *     slot a call reads is first written by that call's own partial kernel, so nothing needs
 *     clearing; but two calls whose kernels may overlap on the GPU (different streams, no
 *     dependency between them) race on the array and give undefined results.  Serialise them.
 */
#define HG_STATIC_SCRATCH_BYTES (8u << 20)
hg_status hg_attn_decode_static(const void* q, const void* k_cache, const void* v_cache, const int32_t* seq_lens,
                                const int32_t* tok_begin, const int32_t* tok_end,
                                const hg_partial_src* host_partials, int32_t n_host_src, float* out, float* lse,
                                void* stream, const hg_attn_desc* desc);

/*
 * Problem description of hg_attn_partial_from_logits (host struct).
 */
typedef struct hg_logits_desc {
    uint32_t struct_size;  /* sizeof(hg_logits_desc) */
    int32_t batch;         /* B */
    int32_t num_q_heads;   /* Hq, a multiple of num_kv_heads */
    int32_t num_kv_heads;  /* Hkv */
    int32_t head_dim;      /* D in {64, 128} */
    int32_t dtype;         /* hg_dtype of the V rows */
    int32_t max_selected;  /* K: row length of logits / v_rows (selected-token slots per sequence) */
    int32_t chunk_tokens;  /* slots per partial, a multiple of 32, at most 1024 */
    int32_t num_chunks;    /* NC >= ceil(K / chunk_tokens): partials per (sequence, head) */
    int32_t* status;       /* dev, optional (present when struct_size covers it): receives HG_DEV_WAIT_TIMEOUT if a
                              bounded on-chip wait of the kernel ran out */
    uint32_t tune;         /* optional (present when struct_size covers it): HG_LOGITS_TUNE_* bits, 0 = defaults */
    uint32_t reserved;     /* 0 */
} hg_logits_desc;

/* hg_logits_desc.tune: which of the two kernels computes the partials (0: the library's choice, the faster one
   for the shape; tests compare the two; both are bit-reproducible) */
#define HG_LOGITS_TUNE_WARP_MMA 1u   /* the contraction on warp-level MMAs (mma.sync), one CTA per chunk */
#define HG_LOGITS_TUNE_TCGEN05 2u    /* the contraction on tcgen05.mma, the accumulator in tensor memory */

/*
 * Softmax partials from host-computed logits and the matching V rows: the device side of the paper's
 * hand-off (Section 4.2, CPU-side support: the host's Logits Calculator sends the logits of its
 * selected tokens, "a compact vector", and the corresponding V vectors; workflow steps 2, 3 and 5).
 * The result plugs into hg_attn_merge as one more source, which stands for concatenating host and
 * device logits and V rows and taking one softmax over them.
 *
 *   logits   dev float [B][Hq][K]      scaled logits s = q.k / sqrt(D) of the selected tokens, natural units;
 *                                      a slot holding -inf weighs nothing for that head
 *   v_rows   dev 16-bit [B][Hkv][K][D] V rows of those tokens, slot for slot; the query heads of a group share
 *                                      their KV head's rows; 16-byte aligned.  Rows of slots at or beyond n_sel[b]
 *                                      are never used, whatever they hold; rows below n_sel[b] must hold finite
 *                                      numbers even where every head's logit is -inf (their weight is zero, and
 *                                      zero times a NaN is not zero)
 *   n_sel    dev int32 [B]             slots in use per sequence (clamped to [0, K])
 *   o_part, m_part, l_part             dev float [B][Hq][NC][D] / [B][Hq][NC]: chunk c covers slots
 *                                      [c * chunk_tokens, (c+1) * chunk_tokens) below n_sel; empty chunks are
 *                                      (m, l, o) = (-inf, 0, 0)
 * Token order and token indices do not matter for the result and are not passed.
 * Every group size runs the P.V product on tensor cores with P as a two-term (hi + lo) 16-bit expansion, fp32
 * accumulation; m is the exact maximum of the chunk's logits, l the fp32 sum of the unrounded weights.
 */
hg_status hg_attn_partial_from_logits(const float* logits, const void* v_rows, const int32_t* n_sel, float* o_part,
                                      float* m_part, float* l_part, void* stream, const hg_logits_desc* desc);

/*
 * Appends the current decode step's K and V rows to the cache (Section 2.1: the new token's K, V are
 * appended before its attention is computed).
 *
 *   k_new, v_new  dev 16-bit [B][Hkv][D], 16-byte aligned
 *   k_cache, v_cache  dev pools (written)
 *   seq_lens      dev int32 [B]: row b goes to position seq_lens[b], then seq_lens[b] += 1
 *   tok_end       dev int32 [B] or NULL: where it equals the old length it grows too (the slice keeps reaching the
 *                 newest token)
 * The page that holds the new position must already be mapped in the block table (page allocation is the
 * caller's); otherwise the row is dropped and *desc->status = HG_DEV_BAD_PAGE.  chunk fields of desc are unused.
 */
hg_status hg_kv_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache, int32_t* seq_lens,
                       int32_t* tok_end, void* stream, const hg_attn_desc* desc);

/*
 * Device half of the Eviction Engine and Token Mapper (Section 4.2, device-side support): moves the oldest
 * tokens of the GPU slice out, least recently generated first.
 *
 * For every sequence the first ne = min(n_evict[b], max_evict, tok_end[b] - tok_begin[b]) tokens of the slice
 * are copied, in token order, to k_out / v_out (dev 16-bit [B][max_evict][Hkv][D] - the token-major layout
 * hg_host_logits reads), ready for one device-to-host copy by the caller.  Then tok_begin[b] += ne, every page
 * that lies wholly below the new beginning is un-mapped (block-table entry -1) and its physical id listed in
 * freed_pages (dev int32 [B][max_freed], -1 padded; n_freed dev int32 [B]; both may be NULL).  The pools are
 * not modified.  desc->block_table is updated in place (it must be writable); with identity paging (NULL)
 * only tok_begin moves.
 * No page is un-mapped whose id cannot be reported: when freed_pages is given and a sequence would free more
 * than max_freed pages, its eviction stops at the first page that does not fit the list - tok_begin[b] moves
 * only to that page's first token and n_freed[b] = max_freed - so read tok_begin back (new minus old) to learn
 * how many rows of k_out / v_out are valid; max_freed >= max_evict / page_size + 1 never truncates.  With
 * freed_pages == NULL every emptied page is un-mapped (the caller keeps its own record).  A sequence whose
 * evicted range meets an unmapped or out-of-pool block-table entry keeps its tok_begin and its block-table
 * row (its rows of k_out / v_out are unspecified) and *desc->status gets HG_DEV_BAD_PAGE.
 */
hg_status hg_kv_evict(const void* k_cache, const void* v_cache, int32_t* tok_begin, const int32_t* tok_end,
                      const int32_t* n_evict, int32_t max_evict, void* k_out, void* v_out, int32_t* freed_pages,
                      int32_t* n_freed, int32_t max_freed, void* stream, const hg_attn_desc* desc);

/*
 * hg_kv_evict in three steps, for an eviction that drains BESIDE the attention of the same decode step instead
 * of in front of it (Section 4.2, device-side support: the Eviction Engine works under memory pressure while
 * decoding goes on; the Token Mapper's ranges are what keeps both sides consistent).
 *
 *   hg_kv_evict_begin   on the attention's stream, before it: decides for every sequence the rows that leave
 *                       (the rule of hg_kv_evict, including its two cut-backs; pass the max_freed that
 *                       hg_kv_evict_finish will be given, 0 if no list is wanted), records them in
 *                       src_begin[b] (the old beginning) and n_moved[b] (dev int32 [B] each) and advances
 *                       tok_begin.  The block table is not touched.  Everything enqueued on this stream afterwards -
 *                       hg_attn_partial, hg_attn_decode - works on the shrunk slice [tok_begin, tok_end).
 *   hg_kv_evict_copy    on a second stream, after an event recorded behind step 1: copies the recorded rows to
 *                       k_out / v_out (layout as in hg_kv_evict; rows beyond n_moved[b] are left alone).  It only
 *                       reads the pools and block-table entries of the rows that leave.
 *   hg_kv_evict_finish  behind the copy (same second stream, or any stream ordered after it): un-maps the pages
 *                       that lie wholly below the new beginning and lists them, as hg_kv_evict does.
 *
 * Why nothing races: attention over the shrunk slice looks up block-table entries only from tok_begin's page on,
 * and step 3 writes only entries of pages wholly below it - the two never touch the same entry, so step 3 needs
 * no ordering against the attention that runs beside it; the page that holds the new beginning stays mapped and
 * is only read by both.  Attention launched BEFORE step 1 (the previous decode step, over the old range) does read
 * the entries step 3 clears: step 1 sits behind it in stream order and steps 2 and 3 wait for step 1's event, which
 * orders them.  A freed page may be handed out again only once step 3 has completed (wait for its stream or an
 * event behind it); until then the rows are still being read.  Results are those of hg_kv_evict, bit for bit.
 */
hg_status hg_kv_evict_begin(int32_t* tok_begin, const int32_t* tok_end, const int32_t* n_evict, int32_t max_evict,
                            int32_t max_freed, int32_t* src_begin, int32_t* n_moved, void* stream,
                            const hg_attn_desc* desc);
hg_status hg_kv_evict_copy(const void* k_cache, const void* v_cache, const int32_t* src_begin, const int32_t* n_moved,
                           int32_t max_evict, void* k_out, void* v_out, void* stream, const hg_attn_desc* desc);
hg_status hg_kv_evict_finish(const int32_t* src_begin, const int32_t* n_moved, int32_t* freed_pages, int32_t* n_freed,
                             int32_t max_freed, void* stream, const hg_attn_desc* desc);

/*
 * Evidence kernel, not part of the attention path: streams the same K and V tiles through the
 * same TMA pipeline as hg_attn_partial and folds them into one 32-bit checksum per work item
 * (sink: dev uint32 [B][Hkv][NC]).  Used to measure the read ceiling of the paged access pattern.
 */
hg_status hg_kv_read_probe(const void* k_cache, const void* v_cache, const int32_t* seq_lens,
                           const int32_t* tok_begin, const int32_t* tok_end, uint32_t* sink, void* stream,
                           const hg_attn_desc* desc);

const char* hg_status_string(hg_status s);
uint32_t hg_version(void);

#ifdef __cplusplus
}
#endif
#endif /* HYBRIDGEN_ATTN_H_ */
