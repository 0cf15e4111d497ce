/*
 * hybridgen_host.h - host-side (CPU) companions of the device library: the pieces of HybridGen's
 * CPU stage that feed hg_attn_partial_from_logits.  Plain C ABI, host pointers only, no CUDA calls;
 * they work on a machine without a GPU.
 *
 *   hg_host_logits            the Logits Calculator (Section 4.2, CPU-side support): scaled logits
 *                             q.k / sqrt(D) of host-resident keys
 *   hg_host_select_topk       Post-QK^T selection (Section 4.3 / 4.5): the K largest scores per row
 *   hg_host_group_scores      a KV head's token scores from its query heads' logits (their maximum)
 *   hg_host_gather_logits     the selected tokens' logits out of the full rows
 *   hg_host_select_positions  a Pre-QK^T, position-based selection (Section 4.5): the first `sinks` and the
 *                             last `window` tokens
 *   hg_host_select_ranked     a Pre-QK^T selection from ranked candidate lists: the first K of each list
 *   hg_host_gather_rows       gathers the selected tokens' V rows into a staging buffer for the transfer
 *   hg_sched_init / _update   the Feedback Scheduler policy (Algorithm 1)
 *   hg_host_tier_*            host memory bound to one NUMA node, the mechanism under the semantic-aware
 *                             placement of Section 4.4 (K rows in CPU DRAM, V rows in a far tier)
 */
#ifndef HYBRIDGEN_HOST_H_
#define HYBRIDGEN_HOST_H_

#include <stddef.h>
#include <stdint.h>

#include "hybridgen_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Layout of the host-resident K (or V) rows: element (b, t, g, d) at
 * b * seq_stride + t * tok_stride + g * head_stride + d, in 16-bit elements. */
typedef struct hg_host_desc {
    uint32_t struct_size;
    int32_t batch;          /* B */
    int32_t num_q_heads;    /* Hq */
    int32_t num_kv_heads;   /* Hkv */
    int32_t head_dim;       /* D, a multiple of 8 */
    int32_t dtype;          /* hg_dtype */
    int32_t max_selected;   /* K: slots per row in idx / logits */
    int32_t num_rows;       /* token rows per sequence behind k_rows / rows; 0 = not stated (gathers then only
                               refuse negative indices) */
    int64_t seq_stride;
    int64_t tok_stride;
    int64_t head_stride;
    float scale;            /* 0 means 1/sqrt(D) */
    int32_t threads;        /* worker threads; 0 means one per available core */
} hg_host_desc;

/*
 * logits[b][h][i] = scale * <q[b][h], K[b][tok_i][h / G]> for slot i < n_sel[b], where tok_i = idx[b][h / G][i]
 * (idx: host int32 [B][Hkv][K]) or tok_i = i when idx is NULL; slots i >= n_sel[b] receive -inf.
 * q: host [B][Hq][D] 16-bit.  Products are exact, accumulation is fp32.
 * Returns HG_ERR_INVALID_ARG for null pointers or a malformed description.
 */
hg_status hg_host_logits(const void* q, const void* k_rows, const int32_t* idx, const int32_t* n_sel, float* logits,
                         const hg_host_desc* desc);

/*
 * For each of `rows` score rows of length `stride` (the first n[r] entries valid): the indices of the
 * min(k, n[r]) largest scores, in ascending index order; ties go to the lower index; NaN scores are
 * never selected.  idx_out: int32 [rows][k], unused slots -1; n_out[r] = number selected.
 */
hg_status hg_host_select_topk(const float* scores, int64_t rows, int64_t stride, const int32_t* n, int32_t k,
                              int32_t* idx_out, int32_t* n_out);

/*
 * Token scores of a KV head for Post-QK^T selection when `group` query heads share it (they share the
 * selected token set too): scores[r][i] = max over the group's rows of logits[r * group + j][i], for
 * i < n[r]; entries from n[r] on are -inf.  logits: [rows * group][stride], scores: [rows][stride].
 * With group = 1 this is a copy.  The paper leaves the sharing rule open; the maximum keeps every token
 * that matters to any head of the group.
 */
hg_status hg_host_group_scores(const float* logits, int64_t rows, int32_t group, int64_t stride, const int32_t* n,
                               float* scores);

/*
 * out[b][h][i] = full[b][h][idx[b][h / G][i]] for i < n_sel[b], -inf beyond: the logits of the chosen
 * tokens, taken from rows that hold the logits of all host tokens (Post-QK^T computes those anyway).
 * full: [B][Hq][full_stride], idx: int32 [B][Hkv][K], out: [B][Hq][K] with K = desc->max_selected.
 * An index outside [0, full_stride) gives -inf.
 */
hg_status hg_host_gather_logits(const float* full, int64_t full_stride, const int32_t* idx, const int32_t* n_sel,
                                float* out, const hg_host_desc* desc);

/*
 * Position-based selection among n_tokens tokens: the first `sinks` and the last `window` of them, at most k
 * (sinks first), ascending.  Returns the number written to idx_out (capacity k).
 */
int32_t hg_host_select_positions(int32_t n_tokens, int32_t sinks, int32_t window, int32_t k, int32_t* idx_out);

/*
 * Pre-QK^T selection from ranked candidate lists (Section 4.5: any predictor - positions, accumulated scores,
 * head importance - reduces to a list of host token indices, most important first).  ranking: host int32
 * [B][Hkv][R], -1 padded at the end.  Every KV head of sequence b takes the first n_out[b] entries of its list,
 * where n_out[b] = min(k, n_host[b], shortest valid prefix among the sequence's heads) - one count per sequence,
 * because the hand-off carries one slot count per sequence.  idx_out: host int32 [B][Hkv][k], the entries taken,
 * then -1.  An entry that is negative or not below n_host[b] ends its list.
 */
hg_status hg_host_select_ranked(const int32_t* ranking, int32_t batch, int32_t num_kv_heads, int32_t r,
                                const int32_t* n_host, int32_t k, int32_t* idx_out, int32_t* n_out);

/*
 * dst[b][g][i][:] = rows[b][idx[b][g][i]][g][:] for i < n_sel[b] (layout of `rows` as in desc); slots beyond
 * n_sel[b] are zero-filled, and so is a slot whose index is negative (the -1 padding of a selection) or, when
 * desc->num_rows is stated, not below it: no row outside the caller's buffer is read.
 * dst: host 16-bit [B][Hkv][K][D].
 */
hg_status hg_host_gather_rows(const void* rows, const int32_t* idx, const int32_t* n_sel, void* dst,
                              const hg_host_desc* desc);

/*
 * Tiered host memory (Section 4.4).  The paper keeps the K rows, which the CPU reads, in CPU DRAM and the
 * V rows, which only ever travel to the GPU, in a slower and larger tier (CXL-attached memory appears to
 * Linux as a NUMA node without CPUs), by binding allocations to nodes.  These calls are that mechanism:
 * page-aligned anonymous memory whose pages may live on `node` only.
 *
 *   hg_host_tier_alloc    bytes > 0, node >= 0.  HG_ERR_INVALID_ARG for a node the machine does not have,
 *                         HG_ERR_UNSUPPORTED where the kernel refuses the binding, HG_OK and *out otherwise.
 *                         The memory is zero-filled on first touch; register it with the CUDA runtime to
 *                         make transfers from it asynchronous.
 *   hg_host_tier_free     ptr and bytes as allocated.
 *   hg_host_tier_node_of  the node on which the page holding ptr lives now; -1 when it has not been touched
 *                         yet or cannot be told.
 *   hg_host_tier_nodes    number of NUMA nodes with memory that are on line (at least 1).
 */
hg_status hg_host_tier_alloc(size_t bytes, int32_t node, void** out);
void hg_host_tier_free(void* ptr, size_t bytes);
int32_t hg_host_tier_node_of(const void* ptr);
int32_t hg_host_tier_nodes(void);

/* Feedback Scheduler (Algorithm 1). */
typedef enum hg_sched_strategy { HG_SCHED_POST_QK = 0, HG_SCHED_PRE_QK = 1 } hg_sched_strategy;

typedef struct hg_sched_state {
    int32_t k;         /* tokens the CPU stage processes */
    int32_t strategy;  /* hg_sched_strategy */
} hg_sched_state;

/* K <- K_min, strategy <- Post-QK^T. */
void hg_sched_init(hg_sched_state* st, int32_t k_min);

/*
 * One step of the policy on the measured stage latencies (any common unit), branch for branch as
 * Algorithm 1 lists them.  If the CPU stage plus the transfer hides behind the GPU stage
 * (t_cpu + t_tx <= t_gpu) K grows by `step` (up to k_max), whichever strategy is in force; otherwise K
 * shrinks by `step` down to k_min, and at k_min the strategy becomes Pre-QK^T.  No branch sets the
 * strategy back to Post-QK^T: within a run the switch is one-way (call hg_sched_init to start over), so
 * latencies that hover around the balance point move K up and down by one step and never flip the
 * strategy back and forth.
 */
void hg_sched_update(hg_sched_state* st, double t_gpu, double t_cpu, double t_tx, int32_t k_min, int32_t k_max,
                     int32_t step);

#ifdef __cplusplus
}
#endif
#endif /* HYBRIDGEN_HOST_H_ */
