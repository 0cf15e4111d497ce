// Split-KV decode attention partials over a paged 16-bit KV pool (sm_100a).
//
// A work item is (sequence b, KV head g [, block of 8 or 16 query heads], chunk c).  Persistent CTAs take
// items from the list of non-empty items, dynamically through a global counter when the caller
// provides one, else round-robin; the producer warp is the only scheduler, and every filled stage
// carries a descriptor telling the consumers what it holds.  Within a CTA the producer streams, per
// step of 64 tokens (128 at D = 64: two tile pairs), the K tile and the V tile of the item (64 x D each) from HBM into one stage of a
// shared-memory ring with TMA tensor loads - one 5-D box per (page, tensor), 128-byte swizzled - and
// runs ahead across item boundaries, so the ring never drains between items.  Four consumer warps
// each own 16 token rows of every tile and keep a private online-softmax state (running max,
// exp-sum, un-normalised output); the states are merged once per item, using the item's last stage
// as scratch before it is handed back to the producer.  The logits never leave the chip.
//
//   MODE_MHA    one query head per KV head: dot products on CUDA cores, fp32 throughout.
//   MODE_GQA    up to 8 query heads share the KV head: S^T = K q^T and O^T = V^T P^T on warp-level
//               tensor-core MMAs (tokens are the M dimension, heads the N dimension, nothing padded
//               for a group of 8).  P is fed as hi + lo 16-bit terms, so its rounding error is ~2^-17
//               (bf16) / ~2^-22 (fp16) instead of one 16-bit ulp.
//   MODE_GQA2   groups of more than 8 query heads: items of 16 heads, i.e. two such head blocks that share
//               every K and V fragment read from the tile (their query rows come straight from global memory,
//               the second block's epilogue state parks in the warp's V rows).
//   MODE_PROBE  same loads, no attention math: folds the slice's bytes into a checksum.
//
// With p.persistent == 0 the grid is (NC, Hkv * head_blocks, B) and every CTA handles the one item
// its block index names (used for batches or chunks too large for the in-kernel item scan).
//
// Why the stage is a K+V pair and the box a whole page: issuing one TMA tensor load costs the
// producer ~250 cycles plus ~50 per further lane of the same instruction, and every mbarrier
// hand-shake costs another few hundred; at ~50 GB/s per SM that only works if each producer
// iteration moves tens of KB.
#pragma once

#include "hg_device.cuh"

namespace hg {

constexpr int TILE_T = 64;             // tokens per tile
constexpr int CONSUMER_WARPS = 4;
constexpr int CONSUMER_THREADS = CONSUMER_WARPS * 32;
constexpr int THREADS = CONSUMER_THREADS + 32;
constexpr int MAX_STAGES = 8;
constexpr int MAX_CHUNK_PAGES = 512;       // chunk_tokens / page_size, any schedule
constexpr int PERSIST_CHUNK_PAGES = 256;   // ... for the persistent schedule (page ids are double-buffered)
constexpr int PERSIST_MAX_BATCH = 1024;    // sequences the in-kernel item scan handles (its table is 4 bytes each; two CTAs
                                           // of three 34 KB stages leave an SM about 2 KB of shared memory to spare)

constexpr int RANGE_CACHE = 128;           // sequences whose slice bounds are kept in shared memory

enum { MODE_MHA = 0, MODE_GQA = 1, MODE_PROBE = 2, MODE_GQA2 = 3 };   // GQA2: items of 16 query heads (two MMA head blocks)

// Division of a non-negative 31-bit number by a launch constant: n / d = umulhi(n, mul) >> shift with
// mul = ceil(2^(31 + s) / d), s = ceil(log2 d), shift = s - 1 (exact for n < 2^31); d = 1 is flagged by mul = 0.
// The producer warp divides several times per work item; a hardware-less 32-bit division costs it ~100 cycles each.
struct FastDiv {
    uint32_t mul, shift;
};
__device__ __forceinline__ int fast_div(int n, FastDiv f) {
    return f.mul ? (int)(__umulhi((uint32_t)n, f.mul) >> f.shift) : n;
}

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
    int persistent;
    int test_stall;           // HG_FLAG_TEST_STALL: the producer never fills a stage
    int sparse_empty;         // HG_FLAG_SPARSE_EMPTY: empty chunk slots get m and l only, their o rows stay untouched
    int pdl_wait;             // launched as a programmatic dependent: wait for the preceding kernel before using any input
    int spec_prefetch;        // stages of the CTA's guessed first item to request into the L2 while waiting (0: none)
    int32_t* sched;           // two zeroed words: [0] hands out items dynamically, [1] counts the CTAs that are done
                              // drawing (NULL: round-robin)
    float scale_log2;         // logit scale * log2(e)
    FastDiv div_C, div_Hkv;   // division by chunk_tokens and by the number of KV heads
#ifdef HG_TRACE
    long long* trace;         // development builds only: 8 timestamps / counters per CTA
#endif
};

#ifdef HG_TRACE
#define HG_TRACE_AT(slot) do { if (p.trace) p.trace[(size_t)blockIdx.x * 8 + (slot)] = (long long)global_timer_ns(); } while (0)
#define HG_TRACE_SET(slot, v) do { if (p.trace) p.trace[(size_t)blockIdx.x * 8 + (slot)] = (long long)(v); } while (0)
#else
#define HG_TRACE_AT(slot) do { } while (0)
#define HG_TRACE_SET(slot, v) do { } while (0)
#endif

struct Control {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t cbar;                       // barrier among the consumer warps (one arrival per warp)
    int2 sdesc[MAX_STAGES];              // what a filled stage holds: x = item index (-1: no more work), y = tile in item
                                         // (low 16 bits) and, above them, one bit per box of the stage's K tiles that
                                         // was NOT loaded although the item has tokens in it (a bad block-table entry)
    int abort_flag;
    int pages[MAX_CHUNK_PAGES];          // persistent schedule: two buffers, at 0 and at MAX_CHUNK_PAGES / 2
    float red_m[2][64];                  // per-warp running maxima / exp-sums of an item (4 warps x up to 16 heads),
    float red_l[2][64];                  // double-buffered by item parity
    int scan[8];                         // per-warp totals of the set-up scan
    int cum[PERSIST_MAX_BATCH + 1];      // cum[b] = number of items of sequences < b
    int2 rng[RANGE_CACHE];               // clamped slices [tb, te) of the first sequences (all of them in a usual batch):
                                         // the producer decodes an item without going back to global memory
};
static_assert(PERSIST_CHUNK_PAGES <= MAX_CHUNK_PAGES / 2, "page-id double buffer");

// One work item, decoded identically by the producer and by every consumer warp.
struct Item {
    int b, y, c;        // sequence, KV head * head_blocks + head block, chunk slot
    int lo, hi;         // token range
    int tile0, ntiles;  // 64-token tiles covering it
};

// Tokens a sequence's row of the block table can address.
__device__ __forceinline__ int table_reach(const PartialParams& p) {
    return (int)min((long long)p.max_pages << p.page_shift, (long long)INT32_MAX);
}

// Clamped slice [tb, te) of sequence b and its number of chunk slots in use.  The slice also ends where the
// block table's row ends: tokens beyond it have no page to be read from (range_beyond_table() reports them).
__device__ __forceinline__ int seq_chunks(const PartialParams& p, int b, int& tb, int& te) {
    tb = max(p.tok_begin[b], 0);
    te = min(min(p.tok_end[b], p.seq_lens[b]), table_reach(p));
    if (te <= tb) return 0;
    return min(fast_div(te + p.C - 1, p.div_C) - fast_div(tb, p.div_C), p.NC);
}

// Chunk slots in use by a clamped slice [tb, te).
__device__ __forceinline__ int chunks_of(const PartialParams& p, int tb, int te) {
    return te <= tb ? 0 : min(fast_div(te + p.C - 1, p.div_C) - fast_div(tb, p.div_C), p.NC);
}

// True when sequence b's slice reaches past the last page its block-table row can name.
__device__ __forceinline__ bool range_beyond_table(const PartialParams& p, int b) {
    return min(p.tok_end[b], p.seq_lens[b]) > table_reach(p) && max(p.tok_begin[b], 0) < min(p.tok_end[b], p.seq_lens[b]);
}

__device__ __forceinline__ void set_range(const PartialParams& p, Item& it, int tb, int te) {
    const int first = fast_div(tb, p.div_C);
    it.lo = max((first + it.c) * p.C, tb);
    it.hi = min((first + it.c + 1) * p.C, te);
    it.tile0 = it.lo / TILE_T;
    it.ntiles = it.hi > it.lo ? (it.hi + TILE_T - 1) / TILE_T - it.tile0 : 0;
}

// Item i of the persistent schedule: items are ordered by (b, c, y) - within a sequence the KV heads vary fastest - or,
// for groups of more than 8 query heads, by (b, KV head, c, head block).  Only the producer decodes (it looks ahead, so the
// three range loads are off the critical path); consumers get the decoded item with the item's first stage.
__device__ __forceinline__ Item decode_item(const PartialParams& p, const Control& ctl, int i) {
    int lo = 0, hi = p.B;                 // largest b with cum[b] <= i
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (ctl.cum[mid] <= i) lo = mid; else hi = mid;
    }
    Item it;
    it.b = lo;
    int tb, te, nc;
    if (lo < RANGE_CACHE) { tb = ctl.rng[lo].x; te = ctl.rng[lo].y; nc = max(chunks_of(p, tb, te), 1); }
    else nc = max(seq_chunks(p, lo, tb, te), 1);
    const int r = i - ctl.cum[lo];
    if (p.head_blocks == 1) {
        it.c = fast_div(r, p.div_Hkv);    // KV heads vary fastest: CTAs that run side by side read the same pages
        it.y = r - it.c * p.Hkv;
    } else {
        // groups of more than 8 query heads: the head blocks of one (KV head, chunk) sit next to each other in the
        // order, so they are taken at about the same time and the second reader finds part of the tiles in L2
        const int per_g = nc * p.head_blocks;
        const int g = r / per_g, rem = r - g * per_g;
        it.c = rem / p.head_blocks;
        it.y = g * p.head_blocks + (rem - it.c * p.head_blocks);
    }
    set_range(p, it, tb, te);
    return it;
}

// (Register budget: two CTAs per SM are what the shared memory allows; the group-query kernel with items of 8 heads is
// held to the registers of three per SM - 128 instead of 163, nothing spilled, the tile loop is not on the critical
// path - so that CTAs of a kernel launched as a dependent find room beside it earlier.)
template <int D, bool BF16, int MODE>
__global__ void __launch_bounds__(THREADS, MODE == MODE_GQA ? 3 : 2) partial_kernel(const __grid_constant__ CUtensorMap tmK,
                                                          const __grid_constant__ CUtensorMap tmV,
                                                          const PartialParams p) {
    constexpr int HALVES = D / 64;
    constexpr int TILE_BYTES = TILE_T * D * 2;
    constexpr int Q_BYTES = 8 * D * 2;            // the item's query rows (up to 8 heads), present in an item's first stage
    constexpr int SUB = 128 / D;                  // 64-token tiles per stage: a stage is 32 KB of K and V at either head dim,
    constexpr int PAIR_BYTES = 2 * TILE_BYTES;    // so the per-stage hand-shakes cost the same per byte (K tile, V tile)
    constexpr int STAGE_BYTES = SUB * PAIR_BYTES + Q_BYTES;   // SUB x (K tile, V tile), q
    constexpr int NV = 8 * HALVES;     // MHA: d-components owned by a lane
    constexpr int KSTEPS = D / 16;     // GQA: 16-wide steps along d
    constexpr float LN2 = 0.6931471805599453f;
    constexpr bool GQA = MODE == MODE_GQA || MODE == MODE_GQA2;
    constexpr int NB = MODE == MODE_GQA2 ? 2 : 1;        // MMA head blocks (8 query heads each) per item
    constexpr int HPI = 8 * NB;                          // query heads per item
    const float NEG_INF = __int_as_float(0xff800000);

    extern __shared__ uint8_t smem_raw[];
    __shared__ Control ctl;
    __shared__ Item sitem[MAX_STAGES];   // the decoded item, written by the producer with the item's first stage
    const uint32_t stage0 = (smem_u32(smem_raw) + 1023u) & ~1023u;   // the swizzle pattern is anchored at 1024 bytes
    uint8_t* const stage0_ptr = smem_raw + (stage0 - smem_u32(smem_raw));

#if __CUDA_ARCH__ >= 900
    cudaTriggerProgrammaticLaunchCompletion();   // a dependent merge launch may be scheduled while this grid drains
#endif
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Y = p.Hkv * p.head_blocks;
    if (tid == 0) HG_TRACE_AT(0);

    // ---- set-up that touches no input: barriers, tensor-map prefetch ------------------------------------
    if (tid == CONSUMER_THREADS) {
        prefetch_tensormap(&tmK);                    // the descriptors are on their way long before the first load
        prefetch_tensormap(&tmV);
    }
    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&ctl.full[s], 1);
            mbar_init(&ctl.empty[s], CONSUMER_WARPS);
        }
        mbar_init(&ctl.cbar, CONSUMER_WARPS);
        ctl.abort_flag = 0;
        fence_barrier_init();
    }
    // Item counts per sequence for the persistent schedule: cum[b+1] = sum_{b' <= b} nc_b' * Y.  Every thread takes a
    // contiguous block of sequences, a warp scan, then the warps' totals through shared memory.  `report`: flag
    // slices that reach past their block-table row.
    auto scan_items = [&](bool report) {
        const int per = (p.B + THREADS - 1) / THREADS;
        const int b0 = min(p.B, tid * per), b1 = min(p.B, b0 + per);
        int sum = 0;
        bool beyond = false;
        for (int b = b0; b < b1; ++b) {
            int tb, te;
            sum += seq_chunks(p, b, tb, te) * Y;
            beyond |= range_beyond_table(p, b);
            if (b < RANGE_CACHE) ctl.rng[b] = make_int2(tb, te);
        }
        if (report && beyond && p.status && blockIdx.x == 0) atomicOr(p.status, HG_DEV_RANGE);
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) ctl.scan[warp] = incl;
        __syncthreads();
        int run = incl - sum;
        for (int w2 = 0; w2 < warp; ++w2) run += ctl.scan[w2];
        if (tid == 0) ctl.cum[0] = 0;
        for (int b = b0; b < b1; ++b) {
            int tb, te;
            run += seq_chunks(p, b, tb, te) * Y;
            ctl.cum[b + 1] = run;
        }
        __syncthreads();
    };

#if __CUDA_ARCH__ >= 900
    if (p.pdl_wait) {
        // Launched while the kernel before it in the stream is still running (its last CTAs, or a merge, are finishing).
        // Nothing that kernel may have written is USED before the wait below returns; but the time is not wasted:
        // on a guess at this CTA's first work item - the ranges and the block table as they look right now, which is
        // what they will be unless that kernel is the one changing them - the item's first K and V boxes are requested
        // into the L2.  These are hints: every index is bounds-checked, nothing is written, no result depends on what
        // was read here, and everything is read again, for real, after the wait.
        if (p.spec_prefetch && p.persistent) {
            scan_items(false);
            if (warp == CONSUMER_WARPS && (int)blockIdx.x < ctl.cum[p.B]) {
                const Item it = decode_item(p, ctl, (int)blockIdx.x);
                const int rsh = min(p.page_shift, 6), Rr = 1 << rsh, nb = TILE_T >> rsh;
                const int j = lane & (nb - 1), isv = (lane >> (6 - rsh)) & 1, sub = lane >> (7 - rsh);
                const int g = it.y / p.head_blocks;
                for (int t = 0; t < it.ntiles && t < p.spec_prefetch * SUB; t += SUB) {
                    const int t0j = (it.tile0 + t + sub) * TILE_T + j * Rr;
                    if (sub < SUB && t + sub < it.ntiles && t0j < it.hi && t0j + Rr > it.lo) {
                        const int pg = t0j >> p.page_shift;
                        int phys = -1;
                        if (pg >= 0 && pg < p.max_pages)
                            phys = p.block_table ? __ldg(p.block_table + (size_t)it.b * p.max_pages + pg) : it.b * p.max_pages + pg;
                        if (phys >= 0 && phys < p.num_pages && g >= 0 && g < p.Hkv)
                            tma_prefetch_5d(isv ? &tmV : &tmK, 0, t0j & (p.page_size - 1), 0, g, phys);
                    }
                }
            }
            __syncthreads();                 // the guess is done with the tables the real scan is about to rewrite
        }
        cudaGridDependencySynchronize();
    }
#endif

    // Loads whose answers are needed a little later are issued first, so that their round trips overlap the
    // scan below: the status word (a wait that timed out earlier in this call, or a word the caller left set,
    // means: do not queue behind it), and this CTA's second work item (its first is its own block index).
    const int32_t status_at_entry = p.status ? *reinterpret_cast<volatile int32_t*>(p.status) : HG_DEV_OK;
    int early_request = 0;
    if (tid == CONSUMER_THREADS && p.persistent && p.sched && !p.test_stall) early_request = atomicAdd(p.sched, 1);   // (raw ticket)

    // ---- for the persistent schedule the item counts per sequence -------------------------------------------
    int n_items = 1, item_step = 1, item_first = 0;
    if (p.persistent) {
        scan_items(true);
        n_items = ctl.cum[p.B];
        // use only as many CTAs as keeps every CTA's item count equal (+-1); the others only help with the
        // empty slots below
        const int rounds = (n_items + (int)gridDim.x - 1) / (int)gridDim.x;
        item_step = rounds > 0 ? (n_items + rounds - 1) / rounds : 1;
        item_first = blockIdx.x;

        // (CTAs beyond the round-robin width, or any CTA when there is no item at all, still help with the empty
        // chunk slots below before they leave)
    } else {
        if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0 && p.status && range_beyond_table(p, blockIdx.z)) atomicOr(p.status, HG_DEV_RANGE);
        __syncthreads();
    }
    if (status_at_entry & HG_DEV_WAIT_TIMEOUT) return;   // checked only now: its load overlapped the scan's loads
    if (tid == 0) HG_TRACE_AT(1);

    volatile int* abort_flag = &ctl.abort_flag;
    auto get_item = [&](int i) -> Item {
        if (p.persistent) return decode_item(p, ctl, i);
        Item it;
        it.b = blockIdx.z; it.y = blockIdx.y; it.c = blockIdx.x;
        int tb, te;
        seq_chunks(p, it.b, tb, te);
        if (te <= tb) { it.lo = it.hi = it.tile0 = it.ntiles = 0; } else set_range(p, it, tb, te);
        return it;
    };

    if (!p.persistent) {
        // this CTA's only item may be an empty chunk slot: neutral element, nothing to stream
        const Item it = get_item(0);
        if (it.ntiles == 0) {
            if constexpr (MODE == MODE_PROBE) {
                if (tid == 0) p.sink[((size_t)it.b * p.Hkv + it.y) * p.NC + it.c] = 0u;
            } else {
                const int hb = it.y % p.head_blocks, g = it.y / p.head_blocks;
                const int nh = GQA ? min(HPI, p.G - hb * HPI) : 1;
                const int hq0 = GQA ? g * p.G + hb * HPI : g;
                if (!p.sparse_empty)
                    for (int i = tid; i < nh * D; i += THREADS)
                        p.o_part[(((size_t)it.b * p.Hq + hq0 + i / D) * p.NC + it.c) * D + i % D] = 0.f;
                if (tid < nh) {
                    p.m_part[((size_t)it.b * p.Hq + hq0 + tid) * p.NC + it.c] = NEG_INF;
                    p.l_part[((size_t)it.b * p.Hq + hq0 + tid) * p.NC + it.c] = 0.f;
                }
            }
            return;
        }
    }

    // ---- tile geometry in shared memory ---------------------------------------------------------------
    // A tile is 64/R boxes of R token rows (R = min(page_size, 64)); a box is [half][row][128 bytes], the
    // 16-byte chunks of a row XOR-swizzled with (row & 7).
    const int rshift = min(p.page_shift, 6);
    const int R = 1 << rshift;
    const uint32_t half_stride = 128u << rshift;
    const uint32_t box_bytes = (uint32_t)(HALVES * 128) << rshift;
    auto row_off = [&](int r) -> uint32_t { return (uint32_t)(r >> rshift) * box_bytes + (uint32_t)(r & (R - 1)) * 128u; };

    const int row0 = warp * 16;                  // a consumer warp's rows within every tile
    const int gi = lane >> 3, li = lane & 7;     // MHA: 8 lanes share a token row; 4 row groups per warp
    const int quad = lane >> 2, tq = lane & 3;   // GQA: MMA fragment coordinates

    if (warp == CONSUMER_WARPS) {
        // =============================== producer warp ===============================
        const uint64_t policy = l2_evict_first_policy();
        const int nbox = TILE_T >> rshift;           // boxes per tile: 4, 2 or 1
        const int j = lane & (nbox - 1);             // this lane's box
        const int isv = (lane >> (6 - rshift)) & 1;  // 0: K tile, 1: V tile
        const int sub = lane >> (7 - rshift);        // which of the stage's tiles (lanes with sub >= SUB idle)
        constexpr int PER_LANE = PERSIST_CHUNK_PAGES / 32;
        const bool dynamic = p.persistent && p.sched != nullptr;

        // block-table entry of logical page pg of the item's sequence if the page overlaps [lo, hi), else -2
        // (the value is only loaded here; check_page() validates it once it is needed)
        auto lookup = [&](const Item& it, int pg) -> int {
            if ((pg << p.page_shift) < it.hi && ((pg + 1) << p.page_shift) > it.lo && pg < p.max_pages)
                return p.block_table ? __ldg(p.block_table + (size_t)it.b * p.max_pages + pg) : it.b * p.max_pages + pg;
            return -2;                                   // no token of the item on this page
        };
        auto check_page = [&](int phys) -> int {
            if (phys == -2) return -1;
            if (phys < 0 || phys >= p.num_pages) {
                if (p.status) atomicOr(p.status, HG_DEV_BAD_PAGE);
                return -1;
            }
            return phys;
        };
        auto first_page = [&](const Item& it) { return (it.tile0 * TILE_T) >> p.page_shift; };
        auto num_pages_of = [&](const Item& it) {
            return it.ntiles ? (((it.tile0 + it.ntiles) * TILE_T - 1) >> p.page_shift) + 1 - first_page(it) : 0;
        };
        // Index of the k-th item this CTA takes.  With the dynamic schedule lane 0 holds the counter's answer
        // in `raw` until it is needed, so that the atomic's round trip overlaps the current item's loads.
        // (dynamic schedule: every CTA starts with the item of its own block index, the counter hands out
        // the items from gridDim.x on)
        // (With the dynamic schedule request() hands back the counter's raw ticket and nothing is computed from it
        // until settle(): an instruction that depends on the atomic's answer would stall the warp, which issues in
        // order, for the whole round trip to the L2 - a couple of thousand cycles under load.)
        auto request = [&](int k) -> int {
            if (!p.persistent) return k == 0 ? 0 : n_items;
            if (dynamic) {
                if (k == 0) return (int)blockIdx.x;
                if (k == 1) return early_request;
                int raw = 0;
                if (lane == 0) raw = atomicAdd(p.sched, 1);
                return raw;
            }
            return (int)blockIdx.x < item_step ? (int)blockIdx.x + k * item_step : n_items;   // round-robin over item_step CTAs
        };
        auto settle = [&](int raw) -> int { return dynamic ? (int)gridDim.x + __shfl_sync(0xffffffffu, raw, 0) : raw; };

#ifdef HG_TRACE
        long long trace_wait = 0, trace_look = 0;
        const long long trace_c0 = clock64();
#endif
        int s = 0, issued = 0, k = 0;                // ring position, stages armed so far, items taken so far
        uint32_t ph = 0;
        bool alive = true;
        int i_cur = p.test_stall ? n_items : request(0);
        int raw_nxt = request(1);
        Item cur;
        if (i_cur < n_items) {                       // page ids of the first item
            cur = get_item(i_cur);
            const int page0 = first_page(cur), npages = num_pages_of(cur);
            for (int i = lane; i < npages && i < MAX_CHUNK_PAGES; i += 32) ctl.pages[i] = check_page(lookup(cur, page0 + i));
            __syncwarp();
        }
        while (i_cur < n_items && alive) {
#ifdef HG_TRACE
            if (p.trace && lane == 0 && k < 64) {
                long long* tl = p.trace + (size_t)gridDim.x * 8 + ((size_t)blockIdx.x * 64 + k) * 2;
                tl[0] = (long long)global_timer_ns(); tl[1] = issued;
            }
#endif
            const int page0 = first_page(cur);
            const int* const pages = &ctl.pages[(k & 1) * (MAX_CHUNK_PAGES / 2)];
            // the next item (its index was requested one item ago) is looked at the first time this item's loads have
            // to wait for a ring slot (at the item's end at the latest): the request for the item after it goes out, and
            // the next item's page ids start loading (they are parked in shared memory once this item's loads have all
            // been issued)
            int i_nxt = n_items;
            bool has_next = false;
            Item nxt = cur;
            int nxt_ids[PER_LANE];
            int nxt_npages = 0;
            auto look_ahead = [&]() {
#ifdef HG_TRACE
                const long long tl0 = clock64();
#endif
                i_nxt = settle(raw_nxt);
                raw_nxt = request(k + 2);
                has_next = i_nxt < n_items;
                if (has_next) {
                    nxt = get_item(i_nxt);
                    const int np0 = first_page(nxt);
                    nxt_npages = min(num_pages_of(nxt), PERSIST_CHUNK_PAGES);
#pragma unroll
                    for (int u = 0; u < PER_LANE; ++u) {
                        const int idx = u * 32 + lane;
                        nxt_ids[u] = -2;
                        if (u * 32 < nxt_npages && idx < nxt_npages) nxt_ids[u] = lookup(nxt, np0 + idx);   // (the first test is warp-uniform)
                    }
                }
#ifdef HG_TRACE
                trace_look += clock64() - tl0;
#endif
            };
            const int g = cur.y / p.head_blocks;
            const int q_heads = GQA ? min(HPI, p.G - (cur.y % p.head_blocks) * HPI) : 1;
            const int q_head0 = GQA ? g * p.G + (cur.y % p.head_blocks) * HPI : g;
            bool looked = false;                                   // the look-ahead for the next item has been done
            for (int it = 0; it < cur.ntiles; it += SUB) {         // one stage = SUB x (K tile + V tile of 64 tokens)
                // Everything that does not need the ring slot comes first, so that a slot that frees up while this is
                // computed is re-armed the moment the wait returns: the time a slot spends neither in flight nor in
                // use comes straight off the bytes in flight (300 cycles more per stage cost the 16-token-page
                // group-query workloads 2 - 2.6 % when it was tried).
                const int t0j = (cur.tile0 + it + sub) * TILE_T + j * R;
                const bool wanted = sub < SUB && it + sub < cur.ntiles && t0j < cur.hi && t0j + R > cur.lo;
                int phys = -1;
                if (wanted) phys = pages[(t0j >> p.page_shift) - page0];
                const uint32_t nvalid = __popc(__ballot_sync(0xffffffffu, phys >= 0));   // K and V boxes
                // boxes the item has tokens in but whose page id was refused: their rows must not enter the result
                const uint32_t missing = __ballot_sync(0xffffffffu, wanted && phys < 0 && !isv) & 0xffffu;
                // (items of 16 heads fetch their query rows themselves: the stage's q slot holds 8)
                const uint32_t qbytes = (MODE != MODE_PROBE && NB == 1 && it == 0) ? (uint32_t)q_heads * D * 2u : 0u;
                uint8_t* const dst = stage0_ptr + (size_t)s * STAGE_BYTES + sub * PAIR_BYTES + isv * TILE_BYTES + j * box_bytes;
                const int c1 = t0j & (p.page_size - 1);

                // the slot: if it is not free yet, the wait is the time for the next item's look-ahead
                int ready = 1;
                if (lane == 0) ready = mbar_try_wait(&ctl.empty[s], ph ^ 1u) ? 1 : 0;
                ready = __shfl_sync(0xffffffffu, ready, 0);
                if (!ready) {
                    if (!looked && it > 0) { look_ahead(); looked = true; }
                    int okw = 1;
#ifdef HG_TRACE
                    const long long tw0 = clock64();
#endif
                    if (lane == 0) okw = mbar_wait(&ctl.empty[s], ph ^ 1u, abort_flag) ? 1 : 0;
#ifdef HG_TRACE
                    trace_wait += clock64() - tw0;
#endif
                    okw = __shfl_sync(0xffffffffu, okw, 0);
                    if (!okw) { alive = false; break; }
                }
                if (lane == 0) {
                    ctl.sdesc[s] = make_int2(i_cur, it | (int)(missing << 16));
                    if (it == 0) sitem[s] = cur;
                    mbar_arrive_expect_tx(&ctl.full[s], nvalid * box_bytes + qbytes);
                }
                // (no warp barrier here: bytes that land before the arrival above is counted cannot complete the phase,
                // the arrival itself is still outstanding)
                if (qbytes && lane == 31)        // the item's query rows travel with its first stage
                    bulk_load(stage0_ptr + (size_t)s * STAGE_BYTES + SUB * PAIR_BYTES,
                              reinterpret_cast<const uint16_t*>(p.q) + ((size_t)cur.b * p.Hq + q_head0) * D, qbytes, &ctl.full[s]);
                if (phys >= 0) tma_load_5d(dst, isv ? &tmV : &tmK, &ctl.full[s], 0, c1, 0, g, phys, policy);
#ifdef HG_PRODUCER_DELAY
                { const long long d0 = clock64(); while (clock64() - d0 < HG_PRODUCER_DELAY) { } }
#endif
                if (issued == 0 && lane == 0) HG_TRACE_AT(2);
                ++issued;
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            }
            if (!alive) break;
            if (!looked) look_ahead();                             // the producer never had to wait during this item
            if (!has_next) break;
            int* const dstp = &ctl.pages[((k + 1) & 1) * (MAX_CHUNK_PAGES / 2)];
#pragma unroll
            for (int u = 0; u < PER_LANE; ++u) {
                const int idx = u * 32 + lane;
                if (idx < nxt_npages) dstp[idx] = check_page(nxt_ids[u]);
            }
            __syncwarp();
            cur = nxt;
            i_cur = i_nxt;
            ++k;
        }
#ifdef HG_TRACE
        if (lane == 0 && p.trace) {
            HG_TRACE_AT(5); HG_TRACE_SET(6, k + 1); HG_TRACE_SET(7, issued);
            long long* ex = p.trace + (size_t)gridDim.x * 8 + (size_t)gridDim.x * 128 + (size_t)blockIdx.x * 8;
            ex[0] = trace_wait; ex[1] = clock64() - trace_c0; ex[7] = trace_look;
        }
#endif
        if (alive && !p.test_stall) {
            // no more work: one last, empty stage tells the consumers
            int okw = 1;
            if (lane == 0) okw = mbar_wait(&ctl.empty[s], ph ^ 1u, abort_flag) ? 1 : 0;
            okw = __shfl_sync(0xffffffffu, okw, 0);
            if (okw && lane == 0) {
                ctl.sdesc[s] = make_int2(-1, 0);
                mbar_arrive_expect_tx(&ctl.full[s], 0u);
            }
        }
        if (dynamic && lane == 0) {
            // This CTA draws no further index.  The last CTA to get here leaves both words of the counter at zero
            // for the next call, which then needs no clearing in front of it.
            __threadfence();
            if (atomicAdd(p.sched + 1, 1) == (int)gridDim.x - 1) {
                p.sched[0] = 0;
                p.sched[1] = 0;
                __threadfence();
            }
        }
        if (*abort_flag && lane == 0) {
            // unwinding: do not leave the CTA while copies into its shared memory may still land
            for (int g2 = max(0, issued - p.stages); g2 < issued; ++g2) {
                int dummy = 0;
                mbar_wait(&ctl.full[g2 % p.stages], (uint32_t)(g2 / p.stages) & 1u, &dummy);
            }
        }
    } else {
        // =============================== consumer warps ===============================
        if (p.persistent) {
            // Empty chunk slots (c >= nc_b) get neutral elements while the first stage is on its way.  The empty
            // slots of one (sequence, head) row are contiguous in all three arrays, so a row is one warp's job: rows
            // are dealt round-robin to the consumer warps of the whole grid and written with full-width stores.
            const int NW = (int)gridDim.x * CONSUMER_WARPS, wg = (int)blockIdx.x * CONSUMER_WARPS + warp;
            const int rows_per_seq = MODE == MODE_PROBE ? p.Hkv : p.Hq;
            for (int r = wg; r < p.B * rows_per_seq; r += NW) {
                const int b = r / rows_per_seq;
                const int nc = (ctl.cum[b + 1] - ctl.cum[b]) / Y;
                const int ne = p.NC - nc;                 // empty slots of this row
                if (ne <= 0) continue;
                const size_t first = (size_t)r * p.NC + nc;
                if constexpr (MODE == MODE_PROBE) {
                    for (int i = lane; i < ne; i += 32) p.sink[first + i] = 0u;
                } else {
                    for (int i = lane; i < ne; i += 32) { p.m_part[first + i] = NEG_INF; p.l_part[first + i] = 0.f; }
                    if (!p.sparse_empty) {
                        float4* o4 = reinterpret_cast<float4*>(p.o_part + first * D);
                        for (int i = lane; i < ne * (D / 4); i += 32) o4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            }
        }
        int cs = 0;                // ring position and phase of the next stage to consume
        uint32_t cph = 0;
        // Barrier among the four consumer warps with a bounded wait (false: give up, the CTA is unwinding).
        uint32_t cphase = 0;
        auto consumer_sync = [&]() -> bool {
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl.cbar);
            const bool ok = warp_wait(&ctl.cbar, cphase, abort_flag);
            cphase ^= 1u;
            return ok;
        };
        // Hands a consumed stage back to the producer.  `wrote` tells that this warp stored to the stage
        // through the generic proxy, which must be ordered before the next TMA write into it.
        auto release = [&](int s, bool wrote) {
            if (wrote) fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl.empty[s]);
        };
        // Scratch of the item epilogue: consumer warp w2 parks its state in the memory of its own 16 K rows of
        // the item's last stage (nobody else reads those rows): 2 KB per 64-element column half; a second block of 8
        // heads goes to its 16 V rows of the same stage.
        auto warp_scratch = [&](int s, int w2, int float_idx) -> float* {
            const int blk = float_idx / (8 * D);         // 0: the warp's K rows, 1 (items of 16 heads): its V rows
            float_idx -= blk * 8 * D;
            return reinterpret_cast<float*>(stage0_ptr + (size_t)s * STAGE_BYTES + (size_t)blk * TILE_BYTES + row_off(16 * w2) +
                                            (uint32_t)(float_idx >> 9) * half_stride) + (float_idx & 511);
        };
        // Waits for the next filled stage; returns its ring position, or -1 when there is no more work (or the
        // CTA is unwinding).  d receives the stage's descriptor.
#ifdef HG_TRACE
        bool traced_first = false;
        long long ctrace_wait = 0, ctrace_c0 = 0, ctrace_epi = 0, ctrace_sync = 0, ctrace_begin = 0, ctrace_park = 0;
#endif
        uint32_t missing = 0u;     // of the stage just received: bit (sub * 2 * boxes per tile + box) = that K/V box is absent
        auto next_stage = [&](int2& d) -> int {
            const int s = cs;
#ifdef HG_TRACE
            const long long tw0 = clock64();
#endif
            if (!warp_wait(&ctl.full[s], cph, abort_flag)) return -1;
#ifdef HG_TRACE
            if (traced_first) ctrace_wait += clock64() - tw0;
            if (tid == 0 && !traced_first) { HG_TRACE_AT(3); }
            if (!traced_first) { traced_first = true; ctrace_c0 = clock64(); }
#endif
            if (++cs == p.stages) { cs = 0; cph ^= 1u; }
            d = ctl.sdesc[s];
            missing = (uint32_t)d.y >> 16;
            d.y &= 0xffff;
            return d.x < 0 ? -1 : s;
        };
        // row r of the stage's tile `sub` sits in a box that was loaded
        auto row_present = [&](int sub, int r) -> bool {
            return !((missing >> (sub * (2 * (TILE_T >> rshift)) + (r >> rshift))) & 1u);
        };

        Item cur;
        cur.b = cur.y = cur.c = cur.lo = cur.hi = cur.tile0 = cur.ntiles = 0;
        int hb = 0, nheads = 1, h0 = 0, par = 1;
        auto begin_item = [&](int s) {
            cur = sitem[s];
            par ^= 1;
            hb = cur.y % p.head_blocks;
            const int g = cur.y / p.head_blocks;
            nheads = GQA ? min(HPI, p.G - hb * HPI) : 1;
            h0 = GQA ? g * p.G + hb * HPI : g;                // first query head of this item
        };

        if constexpr (MODE == MODE_PROBE) {
            uint32_t probe_x = 0u;
            for (;;) {
                int2 d;
                const int s = next_stage(d);
                if (s < 0) break;
                if (d.y == 0) { begin_item(s); probe_x = 0u; }
                for (int sub = 0; sub < SUB && d.y + sub < cur.ntiles; ++sub) {
                const uint32_t base = stage0 + s * STAGE_BYTES + sub * PAIR_BYTES;
                const int tokbase = (cur.tile0 + d.y + sub) * TILE_T;
#pragma unroll
                for (int u = 0; u < 8 * HALVES; ++u) {
                    // K and V: 16 rows x HALVES x 8 chunks each per warp; a quarter-warp reads one 128-byte row segment
                    const int idx = u * 32 + lane;
                    const int r = row0 + (idx >> 3) % 16, hh = ((idx >> 3) / 16) % HALVES, kv = (idx >> 3) / (16 * HALVES);
                    const int t = tokbase + r;
                    if (t >= cur.lo && t < cur.hi && (missing == 0u || row_present(sub, r))) {
                        uint4 v = lds128(base + kv * TILE_BYTES + row_off(r) + hh * half_stride + ((idx & 7) << 4));
                        probe_x ^= v.x ^ v.y ^ v.z ^ v.w;
                    }
                }
                }
                if (d.y + SUB < cur.ntiles) { release(s, false); continue; }
                // item epilogue, with the item's last stage as scratch
#pragma unroll
                for (int o = 16; o; o >>= 1) probe_x ^= __shfl_xor_sync(0xffffffffu, probe_x, o);
                if (lane == 0) ctl.red_l[par][warp] = __uint_as_float(probe_x);
                if (!consumer_sync()) break;
                if (tid == 0)
                    p.sink[((size_t)cur.b * p.Hkv + cur.y) * p.NC + cur.c] =
                        __float_as_uint(ctl.red_l[par][0]) ^ __float_as_uint(ctl.red_l[par][1]) ^
                        __float_as_uint(ctl.red_l[par][2]) ^ __float_as_uint(ctl.red_l[par][3]);
                release(s, false);
            }
        } else if constexpr (MODE == MODE_MHA) {
            // ----------------------- MHA (CUDA cores) -----------------------
            float qf[NV], m_run = NEG_INF, l_run = 0.f, o[NV];
            const int rbase = row0 + gi * 4;                      // this lane group's 4 rows
            uint32_t roff[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) roff[k] = row_off(rbase + k) + (uint32_t)((li ^ ((rbase + k) & 7)) << 4);

            for (;;) {
                int2 d;
                const int s = next_stage(d);
                if (s < 0) break;
                if (d.y == 0) {
                    begin_item(s);
                    const uint32_t qs = stage0 + s * STAGE_BYTES + SUB * PAIR_BYTES;
#pragma unroll
                    for (int hh = 0; hh < HALVES; ++hh) {
                        uint4 raw = lds128(qs + hh * 128 + li * 16);
                        float2 a = unpack2<BF16>(raw.x), bb = unpack2<BF16>(raw.y), cc = unpack2<BF16>(raw.z),
                               dd = unpack2<BF16>(raw.w);
                        qf[hh * 8 + 0] = a.x; qf[hh * 8 + 1] = a.y; qf[hh * 8 + 2] = bb.x; qf[hh * 8 + 3] = bb.y;
                        qf[hh * 8 + 4] = cc.x; qf[hh * 8 + 5] = cc.y; qf[hh * 8 + 6] = dd.x; qf[hh * 8 + 7] = dd.y;
                    }
                    m_run = NEG_INF; l_run = 0.f;
#pragma unroll
                    for (int u = 0; u < NV; ++u) o[u] = 0.f;
                }
                for (int sub = 0; sub < SUB && d.y + sub < cur.ntiles; ++sub) {
                const int tokbase = (cur.tile0 + d.y + sub) * TILE_T;
                bool valid[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int t = tokbase + rbase + k;
                    valid[k] = t >= cur.lo && t < cur.hi && (missing == 0u || row_present(sub, rbase + k));
                }
                const uint32_t kbase = stage0 + s * STAGE_BYTES + sub * PAIR_BYTES, vbase = kbase + TILE_BYTES;

                // ---- K tile: 4 logits per lane group ----
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
#pragma unroll
                    for (int hh = 0; hh < HALVES; ++hh) {
                        uint4 raw = lds128(kbase + roff[k] + hh * half_stride);
                        float2 a = unpack2<BF16>(raw.x), bb = unpack2<BF16>(raw.y), cc = unpack2<BF16>(raw.z),
                               dd = unpack2<BF16>(raw.w);
                        const float* qq = &qf[hh * 8];
                        acc[k] = fmaf(a.x, qq[0], acc[k]); acc[k] = fmaf(a.y, qq[1], acc[k]);
                        acc[k] = fmaf(bb.x, qq[2], acc[k]); acc[k] = fmaf(bb.y, qq[3], acc[k]);
                        acc[k] = fmaf(cc.x, qq[4], acc[k]); acc[k] = fmaf(cc.y, qq[5], acc[k]);
                        acc[k] = fmaf(dd.x, qq[6], acc[k]); acc[k] = fmaf(dd.y, qq[7], acc[k]);
                    }
                }
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
                const float m_new = fmaxf(m_run, mx);
                const float m_safe = (m_new == NEG_INF) ? 0.f : m_new;
                const float corr = fast_exp2(m_run - m_safe);
                float pk[4], psum = 0.f;
#pragma unroll
                for (int k = 0; k < 4; ++k) { pk[k] = fast_exp2(s2[k] - m_safe); psum += pk[k]; }
                l_run = l_run * corr + psum;
                m_run = m_new;

                // ---- V tile: o = o * corr + sum_k p_k V_k ----
#pragma unroll
                for (int u = 0; u < NV; ++u) o[u] *= corr;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
#pragma unroll
                    for (int hh = 0; hh < HALVES; ++hh) {
                        uint4 raw = make_uint4(0u, 0u, 0u, 0u);      // rows outside the slice never enter the sum
                        if (valid[k]) raw = lds128(vbase + roff[k] + hh * half_stride);
                        float2 a = unpack2<BF16>(raw.x), bb = unpack2<BF16>(raw.y), cc = unpack2<BF16>(raw.z),
                               dd = unpack2<BF16>(raw.w);
                        float* oo = &o[hh * 8];
                        oo[0] = fmaf(pk[k], a.x, oo[0]); oo[1] = fmaf(pk[k], a.y, oo[1]);
                        oo[2] = fmaf(pk[k], bb.x, oo[2]); oo[3] = fmaf(pk[k], bb.y, oo[3]);
                        oo[4] = fmaf(pk[k], cc.x, oo[4]); oo[5] = fmaf(pk[k], cc.y, oo[5]);
                        oo[6] = fmaf(pk[k], dd.x, oo[6]); oo[7] = fmaf(pk[k], dd.y, oo[7]);
                    }
                }
                }
                if (d.y + SUB < cur.ntiles) { release(s, false); continue; }

                // ---- item epilogue: merge the 16 row-group states (parked in the item's last stage) ----
                const int slot = warp * 4 + gi;
                if (li == 0) { ctl.red_m[par][slot] = m_run; ctl.red_l[par][slot] = l_run; }
#pragma unroll
                for (int hh = 0; hh < HALVES; ++hh) {
                    float4* dst = reinterpret_cast<float4*>(warp_scratch(s, warp, gi * D + hh * 64 + li * 8));
                    dst[0] = make_float4(o[hh * 8 + 0], o[hh * 8 + 1], o[hh * 8 + 2], o[hh * 8 + 3]);
                    dst[1] = make_float4(o[hh * 8 + 4], o[hh * 8 + 5], o[hh * 8 + 6], o[hh * 8 + 7]);
                }
                if (!consumer_sync()) break;
                if (tid < D) {
                    float M = NEG_INF;
#pragma unroll
                    for (int sidx = 0; sidx < 16; ++sidx) M = fmaxf(M, ctl.red_m[par][sidx]);
                    const float Ms = (M == NEG_INF) ? 0.f : M;     // every page of the item refused: an empty partial
                    float accv = 0.f, lsum = 0.f;
#pragma unroll
                    for (int sidx = 0; sidx < 16; ++sidx) {
                        const float w = fast_exp2(ctl.red_m[par][sidx] - Ms);     // -inf states weigh 0
                        accv = fmaf(w, *warp_scratch(s, sidx >> 2, (sidx & 3) * D + tid), accv);
                        lsum = fmaf(w, ctl.red_l[par][sidx], lsum);
                    }
                    const size_t oslot = ((size_t)cur.b * p.Hq + h0) * p.NC + cur.c;
                    st_global_hint(p.o_part + oslot * D + tid, accv, l2_evict_last_policy());      // the merge reads these lines next
                    if (tid == 0) { p.m_part[oslot] = M * LN2; p.l_part[oslot] = lsum; }
                }
                release(s, true);
            }
        } else {
            // ----------------------- GQA (tensor cores) -----------------------
            // NB blocks of 8 query heads share every K and V fragment loaded from the tile.
            uint32_t qb[NB][KSTEPS][2];  // q^T as the B operand of S^T = K q^T
            float m_run[NB][2], l_run[NB][2], oacc[NB][KSTEPS][4];
            // ldmatrix row addresses for this lane
            const int a_row = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;   // K: matrices (rows, rows+8) x (k lo, k hi)
            const int a_kc = lane >> 4;
            const int v_row = row0 + (lane & 7) + (lane >> 4) * 8;         // V^T: matrices (d lo, d hi) x (tok, tok+8)
            const int v_dc = (lane >> 3) & 1;
            const uint32_t a_off = row_off(a_row), v_off = row_off(v_row);
            // item epilogue: vectors of four parked per (head, lane), see there
            constexpr int V4 = KSTEPS / 2;
            auto park_swz = [](int f, int pair) -> int { return D == 128 ? (f ^ pair) : (f ^ (pair & 1) ^ ((pair >> 1) << 2)); };

            for (;;) {
                int2 d;
                const int s = next_stage(d);
                if (s < 0) break;
#ifdef HG_TRACE
                const long long tb0 = clock64();
#endif
                if (d.y == 0) {
                    begin_item(s);
#ifdef HG_TRACE
                    ctrace_sync += clock64() - tb0;      // (development: the begin_item() part of an item's start)
#endif
                    // b0 = q[head quad][16 ks + 2 tq + {0,1}], b1 = the same + 8; heads past the group read as zero
#pragma unroll
                    for (int nb = 0; nb < NB; ++nb) {
                        const bool live = hb * HPI + nb * 8 + quad < p.G;
                        if constexpr (NB == 1) {
                            const uint32_t qs = stage0 + s * STAGE_BYTES + SUB * PAIR_BYTES + quad * (D * 2);
#pragma unroll
                            for (int ks = 0; ks < KSTEPS; ++ks) {
                                qb[nb][ks][0] = live ? lds32(qs + (ks * 8 + tq) * 4) : 0u;
                                qb[nb][ks][1] = live ? lds32(qs + (ks * 8 + 4 + tq) * 4) : 0u;
                            }
                        } else {
                            // 16 heads do not fit the stage's q slot: each lane reads its 2 x KSTEPS words from global memory
                            const uint32_t* qg = reinterpret_cast<const uint32_t*>(
                                reinterpret_cast<const uint16_t*>(p.q) + ((size_t)cur.b * p.Hq + (live ? h0 + nb * 8 + quad : 0)) * D);
#pragma unroll
                            for (int ks = 0; ks < KSTEPS; ++ks) {
                                qb[nb][ks][0] = live ? __ldg(qg + ks * 8 + tq) : 0u;
                                qb[nb][ks][1] = live ? __ldg(qg + ks * 8 + 4 + tq) : 0u;
                            }
                        }
                        m_run[nb][0] = m_run[nb][1] = NEG_INF; l_run[nb][0] = l_run[nb][1] = 0.f;
#pragma unroll
                        for (int u = 0; u < KSTEPS; ++u) { oacc[nb][u][0] = oacc[nb][u][1] = oacc[nb][u][2] = oacc[nb][u][3] = 0.f; }
                    }
                }
#ifdef HG_TRACE
                if (d.y == 0) ctrace_begin += clock64() - tb0;
#endif
                bool wrote = false;
                for (int sub = 0; sub < SUB && d.y + sub < cur.ntiles; ++sub) {
                const int tokbase = (cur.tile0 + d.y + sub) * TILE_T;
                const int tA = tokbase + row0 + quad, tB = tA + 8;
                const bool vA = tA >= cur.lo && tA < cur.hi && (missing == 0u || row_present(sub, row0 + quad));
                const bool vB = tB >= cur.lo && tB < cur.hi && (missing == 0u || row_present(sub, row0 + quad + 8));
                const bool edge = tokbase < cur.lo || tokbase + TILE_T > cur.hi || missing != 0u;
                wrote |= edge;
                const uint32_t kbase = stage0 + s * STAGE_BYTES + sub * PAIR_BYTES, vbase = kbase + TILE_BYTES;

                if (edge) {
                    // rows outside the slice may hold anything (even NaN patterns): clear this warp's copies in the V tile
                    for (int u = lane; u < 16 * 8 * HALVES; u += 32) {
                        const int r = row0 + (u / (8 * HALVES)), ch = u % (8 * HALVES);
                        const int t = tokbase + r;
                        if (t < cur.lo || t >= cur.hi || !row_present(sub, r)) sts128_zero(vbase + row_off(r) + (ch >> 3) * half_stride + ((ch & 7) << 4));
                    }
                    __syncwarp();
                }

                // ---- S^T (16 tokens x 8 heads per block) ----
                // One head block: all fragment loads are issued before the first MMA, the products accumulate in two
                // independent chains, and the V fragments are requested before the softmax arithmetic, so that the
                // warp (the only one of its CTA on its scheduler) is not held up by one dependent instruction after
                // the other.  Two head blocks already give two independent chains and have no registers to spare.
                float sc[NB][4];
                uint32_t va[NB == 1 ? KSTEPS : 1][4];
                if constexpr (NB == 1) {
                    uint32_t ka[KSTEPS][4];
#pragma unroll
                    for (int ks = 0; ks < KSTEPS; ++ks) {
                        const int ch = 2 * ks + a_kc;   // 16-byte chunk index along d
                        ldmatrix_x4(ka[ks], kbase + a_off + (ch >> 3) * half_stride + (((ch & 7) ^ (a_row & 7)) << 4));
                    }
                    float se[4] = {0.f, 0.f, 0.f, 0.f}, so[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int ks = 0; ks < KSTEPS; ks += 2) {
                        mma_16816<BF16>(se, ka[ks], qb[0][ks][0], qb[0][ks][1]);
                        mma_16816<BF16>(so, ka[ks + 1], qb[0][ks + 1][0], qb[0][ks + 1][1]);
                    }
#pragma unroll
                    for (int mt = 0; mt < KSTEPS; ++mt) {
                        const int ch = 2 * mt + v_dc;
                        ldmatrix_x4_trans(va[mt], vbase + v_off + (ch >> 3) * half_stride + (((ch & 7) ^ (v_row & 7)) << 4));
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i) sc[0][i] = se[i] + so[i];
                } else {
#pragma unroll
                    for (int nb = 0; nb < NB; ++nb) sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
#pragma unroll
                    for (int ks = 0; ks < KSTEPS; ++ks) {
                        const int ch = 2 * ks + a_kc;
                        uint32_t a[4];
                        ldmatrix_x4(a, kbase + a_off + (ch >> 3) * half_stride + (((ch & 7) ^ (a_row & 7)) << 4));
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) mma_16816<BF16>(sc[nb], a, qb[nb][ks][0], qb[nb][ks][1]);
                    }
                }
                float corr[NB][2];
                uint32_t bh0[NB], bh1[NB], bl0[NB], bl1[NB];
                bool moved = false;              // some running maximum of this lane grew: the accumulators need rescaling
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
                    // sc[0], sc[1]: token tA, heads 2tq, 2tq+1 of the block; sc[2], sc[3]: token tB
                    float s2[4];
                    s2[0] = vA ? sc[nb][0] * p.scale_log2 : NEG_INF; s2[1] = vA ? sc[nb][1] * p.scale_log2 : NEG_INF;
                    s2[2] = vB ? sc[nb][2] * p.scale_log2 : NEG_INF; s2[3] = vB ? sc[nb][3] * p.scale_log2 : NEG_INF;
                    float mx[2] = {fmaxf(s2[0], s2[2]), fmaxf(s2[1], s2[3])};
#pragma unroll
                    for (int o = 4; o <= 16; o <<= 1) {
                        mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], o));
                        mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], o));
                    }
                    float msafe[2];
#pragma unroll
                    for (int hc = 0; hc < 2; ++hc) {
                        const float m_new = fmaxf(m_run[nb][hc], mx[hc]);
                        msafe[hc] = (m_new == NEG_INF) ? 0.f : m_new;
                        const bool same = m_new == m_run[nb][hc];
                        corr[nb][hc] = same ? 1.f : fast_exp2(m_run[nb][hc] - msafe[hc]);
                        moved |= !same;
                        m_run[nb][hc] = m_new;
                    }
                    float pr[4];
                    pr[0] = fast_exp2(s2[0] - msafe[0]); pr[1] = fast_exp2(s2[1] - msafe[1]);
                    pr[2] = fast_exp2(s2[2] - msafe[0]); pr[3] = fast_exp2(s2[3] - msafe[1]);
                    l_run[nb][0] = l_run[nb][0] * corr[nb][0] + pr[0] + pr[2];   // per-lane sums over its own two token rows
                    l_run[nb][1] = l_run[nb][1] * corr[nb][1] + pr[1] + pr[3];

                    // P^T as the B operand of O^T += V^T P^T, as hi + lo 16-bit terms
                    const uint32_t hiA = pack2<BF16>(pr[0], pr[1]), hiB = pack2<BF16>(pr[2], pr[3]);
                    const float2 fA = unpack2<BF16>(hiA), fB = unpack2<BF16>(hiB);
                    const uint32_t loA = pack2<BF16>(pr[0] - fA.x, pr[1] - fA.y), loB = pack2<BF16>(pr[2] - fB.x, pr[3] - fB.y);
                    bh0[nb] = movmatrix_trans(hiA); bh1[nb] = movmatrix_trans(hiB);
                    bl0[nb] = movmatrix_trans(loA); bl1[nb] = movmatrix_trans(loB);
                }

                // ---- O^T ----
                // the running maxima settle after an item's first tiles: most tiles need no rescaling at all
                if (__any_sync(0xffffffffu, moved)) {
#pragma unroll
                    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
                        for (int mt = 0; mt < KSTEPS; ++mt) {
                            oacc[nb][mt][0] *= corr[nb][0]; oacc[nb][mt][1] *= corr[nb][1];
                            oacc[nb][mt][2] *= corr[nb][0]; oacc[nb][mt][3] *= corr[nb][1];
                        }
                }
                if constexpr (NB == 1) {
#pragma unroll
                    for (int mt = 0; mt < KSTEPS; ++mt) mma_16816<BF16>(oacc[0][mt], va[mt], bh0[0], bh1[0]);
#pragma unroll
                    for (int mt = 0; mt < KSTEPS; ++mt) mma_16816<BF16>(oacc[0][mt], va[mt], bl0[0], bl1[0]);
                } else {
#pragma unroll
                    for (int mt = 0; mt < KSTEPS; ++mt) {
                        const int ch = 2 * mt + v_dc;
                        ldmatrix_x4_trans(va[0], vbase + v_off + (ch >> 3) * half_stride + (((ch & 7) ^ (v_row & 7)) << 4));
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) mma_16816<BF16>(oacc[nb][mt], va[0], bh0[nb], bh1[nb]);
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) mma_16816<BF16>(oacc[nb][mt], va[0], bl0[nb], bl1[nb]);
                    }
                }
                }
                if (d.y + SUB < cur.ntiles) { release(s, wrote); continue; }

                // ---- item epilogue: merge the 4 warp states (the item's last stage is the scratch) ----
#ifdef HG_TRACE
                const long long te0 = clock64();
#endif
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
                    for (int o = 4; o <= 16; o <<= 1) {
                        l_run[nb][0] += __shfl_xor_sync(0xffffffffu, l_run[nb][0], o);
                        l_run[nb][1] += __shfl_xor_sync(0xffffffffu, l_run[nb][1], o);
                    }
                    if (quad == 0) {
                        const int e = warp * HPI + nb * 8 + 2 * tq;
                        ctl.red_m[par][e] = m_run[nb][0]; ctl.red_m[par][e + 1] = m_run[nb][1];
                        ctl.red_l[par][e] = l_run[nb][0]; ctl.red_l[par][e + 1] = l_run[nb][1];
                    }
                    // This warp's [8 heads][D] of the block into its own rows.  A lane holds 2 x KSTEPS components of
                    // each of its two heads (d = 16 mt + quad and that + 8): they are parked as V4 = KSTEPS / 2 vectors
                    // of four per head, vector quad * V4 + i of the head's D / 4 holding d = 32 i + 8 kk + quad
                    // (kk = 0..3), at an index XOR-ed with the lane's head pair so that the eight lanes of a store
                    // phase hit eight different 16-byte bank groups.
#pragma unroll
                    for (int hsel = 0; hsel < 2; ++hsel) {
                        float4* const head_base = reinterpret_cast<float4*>(warp_scratch(s, warp, (nb * 8 + 2 * tq + hsel) * D));
#pragma unroll
                        for (int i = 0; i < V4; ++i)
                            head_base[park_swz(quad * V4 + i, tq)] =
                                make_float4(oacc[nb][2 * i][hsel], oacc[nb][2 * i][2 + hsel], oacc[nb][2 * i + 1][hsel], oacc[nb][2 * i + 1][2 + hsel]);
                    }
                }
#ifdef HG_TRACE
                ctrace_park += clock64() - te0;
#endif
                if (!consumer_sync()) break;
                // thread -> (head, D/16 components: the parked vectors r and, at D = 128, r + 16 of the head): the four
                // warp states of one head, weighted
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
                    constexpr int PER = D / 16;
                    const int hh = nb * 8 + (tid >> 4), r = tid & 15, pair = (tid >> 4) >> 1;
                    if (hh < nheads) {
                        float mw[CONSUMER_WARPS], M = NEG_INF, lsum = 0.f;
#pragma unroll
                        for (int w2 = 0; w2 < CONSUMER_WARPS; ++w2) { mw[w2] = ctl.red_m[par][w2 * HPI + hh]; M = fmaxf(M, mw[w2]); }
                        const float Ms = (M == NEG_INF) ? 0.f : M;     // every page of the item refused: an empty partial
                        float accv[PER];
#pragma unroll
                        for (int v = 0; v < PER; ++v) accv[v] = 0.f;
#pragma unroll
                        for (int w2 = 0; w2 < CONSUMER_WARPS; ++w2) {
                            const float w = fast_exp2(mw[w2] - Ms);
                            lsum = fmaf(w, ctl.red_l[par][w2 * HPI + hh], lsum);
                            const float4* src = reinterpret_cast<const float4*>(warp_scratch(s, w2, hh * D));
#pragma unroll
                            for (int v4 = 0; v4 < PER / 4; ++v4) {
                                const float4 x = src[park_swz(r + 16 * v4, pair)];
                                accv[v4 * 4 + 0] = fmaf(w, x.x, accv[v4 * 4 + 0]); accv[v4 * 4 + 1] = fmaf(w, x.y, accv[v4 * 4 + 1]);
                                accv[v4 * 4 + 2] = fmaf(w, x.z, accv[v4 * 4 + 2]); accv[v4 * 4 + 3] = fmaf(w, x.w, accv[v4 * 4 + 3]);
                            }
                        }
                        const size_t oslot = ((size_t)cur.b * p.Hq + h0 + hh) * p.NC + cur.c;
                        float* const dst = p.o_part + oslot * D;
                        const uint64_t keep = l2_evict_last_policy();      // the merge reads these lines next
#pragma unroll
                        for (int v4 = 0; v4 < PER / 4; ++v4) {
                            const int f = r + 16 * v4, d0 = 32 * (f % V4) + f / V4;      // component kk of vector f: d0 + 8 kk
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) st_global_hint(dst + d0 + 8 * kk, accv[v4 * 4 + kk], keep);
                        }
                        if (r == 0) { p.m_part[oslot] = M * LN2; p.l_part[oslot] = lsum; }
                    }
                }
                release(s, true);
#ifdef HG_TRACE
                ctrace_epi += clock64() - te0;
#endif
            }
        }
#ifdef HG_TRACE
        if (tid == 0 && p.trace) {
            long long* ex = p.trace + (size_t)gridDim.x * 8 + (size_t)gridDim.x * 128 + (size_t)blockIdx.x * 8;
            ex[2] = ctrace_wait; ex[3] = clock64() - ctrace_c0; ex[4] = ctrace_epi; ex[5] = ctrace_sync; ex[6] = ctrace_begin; ex[0] = ctrace_park;
        }
#endif
    }

    // ---- all roles meet; report a timed-out wait ---------------------------------------------------------
    __syncthreads();
    if (tid == 0) HG_TRACE_AT(4);
    if (*abort_flag && p.status && tid == 0) atomicOr(p.status, HG_DEV_WAIT_TIMEOUT);
}

}  // namespace hg
