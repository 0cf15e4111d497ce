// Host-side companions declared in include/hybridgen_host.h: logits calculator, token selection, row
// gather and the feedback scheduler policy.  No CUDA here.
#include "hybridgen_host.h"

#include <math.h>
#include <string.h>

#include <pthread.h>
#include <stdio.h>
#if defined(__linux__)
#include <sys/mman.h>
#include <sys/syscall.h>
#include <unistd.h>
#endif

#include <algorithm>
#include <atomic>
#include <condition_variable>
#include <functional>
#include <mutex>
#include <limits>
#include <thread>
#include <vector>

#if defined(__x86_64__)
#include <immintrin.h>
#endif

namespace {

inline float half_bits_to_float(uint16_t h) {
    const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1fu, man = h & 0x3ffu, out;
    if (exp == 0) {
        if (man == 0) out = sign;
        else {                                   // subnormal: normalise
            int e = -1;
            do { man <<= 1; ++e; } while (!(man & 0x400u));
            out = sign | ((uint32_t)(127 - 15 - e) << 23) | ((man & 0x3ffu) << 13);
        }
    } else if (exp == 31) out = sign | 0x7f800000u | (man << 13);
    else out = sign | ((exp + 112u) << 23) | (man << 13);
    float f;
    memcpy(&f, &out, 4);
    return f;
}

inline float bf16_bits_to_float(uint16_t h) {
    const uint32_t out = (uint32_t)h << 16;
    float f;
    memcpy(&f, &out, 4);
    return f;
}

#if defined(__x86_64__)
bool have_avx2() {
    static const bool ok = __builtin_cpu_supports("avx2") && __builtin_cpu_supports("fma") && __builtin_cpu_supports("f16c");
    return ok;
}
#endif

// ---- row copies into the transfer buffer ----------------------------------------------------------------------
// The staging buffer is written once and then read by the GPU's copy engine, never by a core: streaming stores
// put the rows in memory without leaving dirty lines in some core's cache for the engine to chase.

#if defined(__x86_64__)
__attribute__((target("avx2"))) void copy_row_stream(void* dst, const void* src, size_t bytes) {
    const __m256i* s = static_cast<const __m256i*>(src);
    __m256i* d = static_cast<__m256i*>(dst);
    for (size_t i = 0; i < bytes / 32; ++i) _mm256_stream_si256(d + i, _mm256_loadu_si256(s + i));
}
#endif

inline void copy_row(void* dst, const void* src, size_t bytes) {
#if defined(__x86_64__)
    if (have_avx2() && bytes % 32 == 0 && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) { copy_row_stream(dst, src, bytes); return; }
#endif
    memcpy(dst, src, bytes);
}

inline void rows_written() {
#if defined(__x86_64__)
    _mm_sfence();                                    // streaming stores are ordered before whatever publishes the buffer
#endif
}

// ---- tiled logits: TILE_T token rows of one KV head against the G query heads that share it ------------
//
// The rows are converted to fp32 once into a small buffer; every head of the group then takes its dot
// products from that buffer with one accumulator per token, and the TILE_T accumulators are summed across
// lanes together (a transposing add tree) so that a head's logits for the tile leave as one vector.

constexpr int TILE_T = 16;
constexpr int MAX_D = 256;

struct TileArgs {
    const uint16_t* rows[TILE_T];   // K rows of the tile (rows past `valid` repeat the last valid one)
    const uint16_t* next[TILE_T];   // the rows the following tile will read: prefetched while this one is converted
    int valid;                      // tokens of the tile that exist
    int D, G;
    bool bf16;
    float scale;
    const float* qf;                // [G][D] fp32 query rows of the group
    float* out;                     // logits of the group's first head at the tile's first token
    int64_t out_stride;             // floats between consecutive heads
};

void tile_scalar(const TileArgs& a) {
    for (int h = 0; h < a.G; ++h)
        for (int t = 0; t < a.valid; ++t) {
            float acc = 0.f;
            const float* q = a.qf + (int64_t)h * a.D;
            for (int d = 0; d < a.D; ++d)
                acc = fmaf(a.bf16 ? bf16_bits_to_float(a.rows[t][d]) : half_bits_to_float(a.rows[t][d]), q[d], acc);
            a.out[h * a.out_stride + t] = a.scale * acc;
        }
}

#if defined(__x86_64__)
// eight accumulators -> one vector holding their eight horizontal sums
__attribute__((target("avx2,fma,f16c"))) inline __m256 hsum8(const __m256* v) {
    const __m256 h01 = _mm256_hadd_ps(v[0], v[1]), h23 = _mm256_hadd_ps(v[2], v[3]);
    const __m256 h45 = _mm256_hadd_ps(v[4], v[5]), h67 = _mm256_hadd_ps(v[6], v[7]);
    const __m256 a = _mm256_hadd_ps(h01, h23), b = _mm256_hadd_ps(h45, h67);
    return _mm256_add_ps(_mm256_permute2f128_ps(a, b, 0x20), _mm256_permute2f128_ps(a, b, 0x31));
}

__attribute__((target("avx2,fma,f16c"))) void tile_avx2(const TileArgs& a) {
    alignas(32) float buf[TILE_T * MAX_D];
    const int D = a.D;
    for (int t = 0; t < TILE_T; ++t) {
        for (int d = 0; d < D; d += 32) _mm_prefetch(reinterpret_cast<const char*>(a.next[t] + d), _MM_HINT_T0);
        for (int d = 0; d < D; d += 8) {
            const __m128i r = _mm_loadu_si128(reinterpret_cast<const __m128i*>(a.rows[t] + d));
            const __m256 f = a.bf16 ? _mm256_castsi256_ps(_mm256_slli_epi32(_mm256_cvtepu16_epi32(r), 16)) : _mm256_cvtph_ps(r);
            _mm256_store_ps(buf + t * D + d, f);
        }
    }
    const __m256 sc = _mm256_set1_ps(a.scale);
    for (int h = 0; h < a.G; ++h) {
        const float* q = a.qf + (int64_t)h * D;
        alignas(32) float res[TILE_T];
        for (int half = 0; half < 2; ++half) {
            __m256 acc[8];
            for (int t = 0; t < 8; ++t) acc[t] = _mm256_setzero_ps();
            const float* b0 = buf + half * 8 * D;
            for (int d = 0; d < D; d += 8) {
                const __m256 qv = _mm256_loadu_ps(q + d);
                for (int t = 0; t < 8; ++t) acc[t] = _mm256_fmadd_ps(_mm256_load_ps(b0 + t * D + d), qv, acc[t]);
            }
            _mm256_store_ps(res + half * 8, _mm256_mul_ps(hsum8(acc), sc));
        }
        float* o = a.out + h * a.out_stride;
        if (a.valid == TILE_T) { _mm256_storeu_ps(o, _mm256_load_ps(res)); _mm256_storeu_ps(o + 8, _mm256_load_ps(res + 8)); }
        else memcpy(o, res, sizeof(float) * a.valid);
    }
}

__attribute__((target("avx512f,avx2,fma,f16c"))) void tile_avx512(const TileArgs& a) {
    alignas(64) float buf[TILE_T * MAX_D];
    const int D = a.D;                                   // a multiple of 16 here
    for (int t = 0; t < TILE_T; ++t) {
        for (int d = 0; d < D; d += 32) _mm_prefetch(reinterpret_cast<const char*>(a.next[t] + d), _MM_HINT_T0);
        for (int d = 0; d < D; d += 16) {
            const __m256i r = _mm256_loadu_si256(reinterpret_cast<const __m256i*>(a.rows[t] + d));
            const __m512 f = a.bf16 ? _mm512_castsi512_ps(_mm512_slli_epi32(_mm512_cvtepu16_epi32(r), 16)) : _mm512_cvtph_ps(r);
            _mm512_store_ps(buf + t * D + d, f);
        }
    }
    const __m256 sc = _mm256_set1_ps(a.scale);
    for (int h = 0; h < a.G; ++h) {
        const float* q = a.qf + (int64_t)h * D;
        __m512 acc[TILE_T];
        for (int t = 0; t < TILE_T; ++t) acc[t] = _mm512_setzero_ps();
        for (int d = 0; d < D; d += 16) {
            const __m512 qv = _mm512_loadu_ps(q + d);
            for (int t = 0; t < TILE_T; ++t) acc[t] = _mm512_fmadd_ps(_mm512_load_ps(buf + t * D + d), qv, acc[t]);
        }
        __m256 half[TILE_T];
        for (int t = 0; t < TILE_T; ++t)
            half[t] = _mm256_add_ps(_mm512_castps512_ps256(acc[t]),
                                    _mm256_castpd_ps(_mm512_extractf64x4_pd(_mm512_castps_pd(acc[t]), 1)));
        alignas(32) float res[TILE_T];
        _mm256_store_ps(res, _mm256_mul_ps(hsum8(half), sc));
        _mm256_store_ps(res + 8, _mm256_mul_ps(hsum8(half + 8), sc));
        float* o = a.out + h * a.out_stride;
        if (a.valid == TILE_T) { _mm256_storeu_ps(o, _mm256_load_ps(res)); _mm256_storeu_ps(o + 8, _mm256_load_ps(res + 8)); }
        else memcpy(o, res, sizeof(float) * a.valid);
    }
}
bool have_avx512() {
    static const bool ok = have_avx2() && __builtin_cpu_supports("avx512f");
    return ok;
}
#endif

using TileFn = void (*)(const TileArgs&);

TileFn pick_tile_fn(int D) {
#if defined(__x86_64__)
    if (D <= MAX_D && D % 16 == 0 && have_avx512()) return tile_avx512;
    if (D <= MAX_D && have_avx2()) return tile_avx2;
#endif
    return tile_scalar;
}

bool desc_ok(const hg_host_desc* d) {
    return d && d->struct_size >= sizeof(hg_host_desc) && d->batch >= 1 && d->num_kv_heads >= 1 && d->num_q_heads >= 1 &&
           d->num_q_heads % d->num_kv_heads == 0 && d->head_dim >= 8 && d->head_dim % 8 == 0 &&
           (d->dtype == HG_DTYPE_F16 || d->dtype == HG_DTYPE_BF16) && d->max_selected >= 1 && d->scale >= 0.f &&
           d->threads >= 0;
}

// Worker threads that outlive a call: starting a thread costs tens of microseconds, a logits call for a
// thousand selected tokens has a few hundred microseconds of work.  The pool grows on demand, is never torn
// down (its threads end with the process) and is forgotten by a forked child, which starts its own.
class Pool {
public:
    // Runs work() on `extra` pool threads and on the caller; returns when all have finished.  A second caller
    // arriving meanwhile is told to fend for itself.
    bool run(int extra, const std::function<void()>& work) {
        std::unique_lock<std::mutex> busy(busy_, std::try_to_lock);
        if (!busy.owns_lock()) return false;
        {
            std::lock_guard<std::mutex> g(mu_);
            while ((int)threads_.size() < extra) threads_.emplace_back([this, id = (int)threads_.size()] { loop(id); });
            work_ = &work; wanted_ = extra; pending_ = extra; ++generation_;
        }
        wake_.notify_all();
        work();
        std::unique_lock<std::mutex> g(mu_);
        done_.wait(g, [this] { return pending_ == 0; });
        work_ = nullptr;
        return true;
    }

private:
    void loop(int id) {
        uint64_t seen = 0;
        for (;;) {
            const std::function<void()>* w;
            {
                std::unique_lock<std::mutex> g(mu_);
                wake_.wait(g, [&] { return generation_ != seen; });
                seen = generation_;
                if (id >= wanted_) continue;
                w = work_;
            }
            (*w)();
            std::lock_guard<std::mutex> g(mu_);
            if (--pending_ == 0) done_.notify_one();
        }
    }
    std::mutex busy_, mu_;
    std::condition_variable wake_, done_;
    std::vector<std::thread> threads_;
    const std::function<void()>* work_ = nullptr;
    int wanted_ = 0, pending_ = 0;
    uint64_t generation_ = 0;
};

std::atomic<Pool*> g_pool{nullptr};

Pool* pool() {
    Pool* p = g_pool.load(std::memory_order_acquire);
    if (p) return p;
    static std::once_flag fork_hook;
    std::call_once(fork_hook, [] { pthread_atfork(nullptr, nullptr, [] { g_pool.store(nullptr); }); });
    Pool* fresh = new Pool;
    if (g_pool.compare_exchange_strong(p, fresh, std::memory_order_acq_rel)) return fresh;
    delete fresh;                                   // another thread was first; no thread had been started in ours
    return p;
}

// Runs fn(i) for i in [0, n) on `threads` workers (0: one per core), the caller being one of them.
template <class F>
void parallel_for(int64_t n, int threads, F fn) {
    int nt = threads > 0 ? threads : (int)std::thread::hardware_concurrency();
    if (nt < 1) nt = 1;
    if (nt > 256) nt = 256;
    if ((int64_t)nt > n) nt = (int)n;
    if (nt <= 1) { for (int64_t i = 0; i < n; ++i) fn(i); return; }
    std::atomic<int64_t> next{0};
    const std::function<void()> work = [&] { for (int64_t i; (i = next.fetch_add(1)) < n;) fn(i); };
    if (pool()->run(nt - 1, work)) return;
    std::vector<std::thread> own;                   // the pool is serving another caller
    for (int t = 1; t < nt; ++t) own.emplace_back(work);
    work();
    for (auto& t : own) t.join();
}

}  // namespace

extern "C" {

hg_status hg_host_logits(const void* q, const void* k_rows, const int32_t* idx, const int32_t* n_sel, float* logits,
                         const hg_host_desc* d) {
    if (!desc_ok(d) || !q || !k_rows || !n_sel || !logits) return HG_ERR_INVALID_ARG;
    const int D = d->head_dim, G = d->num_q_heads / d->num_kv_heads, K = d->max_selected;
    const bool bf16 = d->dtype == HG_DTYPE_BF16;
    const float scale = d->scale > 0.f ? d->scale : 1.0f / sqrtf((float)D);
    const uint16_t* qp = static_cast<const uint16_t*>(q);
    const uint16_t* kp = static_cast<const uint16_t*>(k_rows);
    const int Hq = d->num_q_heads, Hkv = d->num_kv_heads;
    // query rows once as fp32
    std::vector<float> qf((size_t)d->batch * Hq * D);
    for (size_t i = 0; i < qf.size(); ++i) qf[i] = bf16 ? bf16_bits_to_float(qp[i]) : half_bits_to_float(qp[i]);
    const TileFn tile = pick_tile_fn(D);

    // Work items: (sequence, block of tokens, KV heads).  When a token's heads lie next to each other in memory
    // (token-major rows) one item sweeps all heads of its tokens, so that memory is read front to back; with
    // head-major rows every KV head is an item of its own stream.
    const bool token_major = d->head_stride < d->tok_stride;
    const int g_per_item = token_major ? Hkv : 1;
    const int g_items = Hkv / g_per_item;
    // a worker thread costs tens of microseconds to wake: give each at least 256 KB of keys to read
    int64_t key_bytes = 0;
    for (int b = 0; b < d->batch; ++b) key_bytes += (int64_t)std::max(0, std::min(n_sel[b], K)) * Hkv * D * 2;
    int workers = d->threads > 0 ? d->threads : (int)std::thread::hardware_concurrency();
    workers = (int)std::max<int64_t>(1, std::min<int64_t>(workers, key_bytes >> 18));
    // token blocks of up to 256, smaller when that is what it takes to give every worker a few items
    int BLOCK = 256;
    while (BLOCK > TILE_T && (int64_t)d->batch * ((K + BLOCK - 1) / BLOCK) * g_items < 4 * (int64_t)workers) BLOCK /= 2;
    const int blocks = (K + BLOCK - 1) / BLOCK;
    parallel_for((int64_t)d->batch * blocks * g_items, workers, [&](int64_t item) {
        const int gi = (int)(item % g_items);
        const int blk = (int)((item / g_items) % blocks);
        const int b = (int)(item / ((int64_t)g_items * blocks));
        const int n = std::max(0, std::min(n_sel[b], K));
        const int t0 = blk * BLOCK, t1 = std::min(K, t0 + BLOCK);
        const float ninf = -std::numeric_limits<float>::infinity();
        const int g0 = gi * g_per_item, g1 = g0 + g_per_item;
        TileArgs a;
        a.D = D; a.G = G; a.bf16 = bf16; a.scale = scale; a.out_stride = K;
        // tile by tile, and within a tile head by head: with token-major rows that walks each token's row from
        // its first head to its last
        for (int t = t0; t < std::min(t1, n); t += TILE_T) {
            a.valid = std::min(TILE_T, n - t);
            for (int g = g0; g < g1; ++g) {
                const uint16_t* kb = kp + (int64_t)b * d->seq_stride + (int64_t)g * d->head_stride;
                const int32_t* ix = idx ? idx + ((int64_t)b * Hkv + g) * K : nullptr;
                for (int i = 0; i < TILE_T; ++i) {
                    const int tt = t + std::min(i, a.valid - 1);
                    const int tn = std::min(tt + TILE_T, n - 1);
                    a.rows[i] = kb + (int64_t)(ix ? ix[tt] : tt) * d->tok_stride;
                    a.next[i] = kb + (int64_t)(ix ? ix[tn] : tn) * d->tok_stride;
                }
                a.qf = qf.data() + ((size_t)b * Hq + (size_t)g * G) * D;
                a.out = logits + ((int64_t)b * Hq + (int64_t)g * G) * K + t;
                tile(a);
            }
        }
        for (int h = g0 * G; h < g1 * G; ++h)
            for (int t = std::max(t0, n); t < t1; ++t) logits[((int64_t)b * Hq + h) * K + t] = ninf;
    });
    return HG_OK;
}

hg_status hg_host_select_topk(const float* scores, int64_t rows, int64_t stride, const int32_t* n, int32_t k,
                              int32_t* idx_out, int32_t* n_out) {
    if (!scores || !n || !idx_out || rows < 0 || stride < 1 || k < 1) return HG_ERR_INVALID_ARG;
    parallel_for(rows, 0, [&](int64_t r) {
        const float* s = scores + r * stride;
        const int nv = (int)std::max<int64_t>(0, std::min<int64_t>(n[r], stride));
        // value of the k-th largest score (NaN left out), then one pass in index order: everything above it, and of
        // the scores equal to it the lowest indices until k are taken - the same set as sorting by (-score, index)
        std::vector<float> vals;
        vals.reserve(nv);
        for (int i = 0; i < nv; ++i) if (s[i] == s[i]) vals.push_back(s[i]);
        const int take = std::min<int>(k, (int)vals.size());
        int32_t* out = idx_out + r * k;
        int w = 0;
        if (take == (int)vals.size()) {
            for (int i = 0; i < nv; ++i) if (s[i] == s[i]) out[w++] = i;
        } else if (take > 0) {
            std::nth_element(vals.begin(), vals.begin() + (take - 1), vals.end(), std::greater<float>());
            const float kth = vals[take - 1];
            int above = 0;
            for (int i = 0; i < nv; ++i) above += s[i] > kth;
            int ties = take - above;                           // how many scores equal to kth still fit
            for (int i = 0; i < nv && w < take; ++i) {
                if (s[i] > kth) out[w++] = i;
                else if (s[i] == kth && ties > 0) { out[w++] = i; --ties; }
            }
        }
        for (int i = w; i < k; ++i) out[i] = -1;
        if (n_out) n_out[r] = take;
    });
    return HG_OK;
}

hg_status hg_host_group_scores(const float* logits, int64_t rows, int32_t group, int64_t stride, const int32_t* n,
                               float* scores) {
    if (!logits || !n || !scores || rows < 0 || group < 1 || stride < 1) return HG_ERR_INVALID_ARG;
    const float ninf = -std::numeric_limits<float>::infinity();
    parallel_for(rows, 0, [&](int64_t r) {
        const int64_t nv = std::max<int64_t>(0, std::min<int64_t>(n[r], stride));
        float* out = scores + r * stride;
        const float* in = logits + r * group * stride;
        for (int64_t i = 0; i < nv; ++i) out[i] = in[i];
        for (int j = 1; j < group; ++j) {
            const float* row = in + (int64_t)j * stride;
            for (int64_t i = 0; i < nv; ++i) out[i] = row[i] > out[i] || out[i] != out[i] ? row[i] : out[i];
        }
        for (int64_t i = nv; i < stride; ++i) out[i] = ninf;
    });
    return HG_OK;
}

hg_status hg_host_gather_logits(const float* full, int64_t full_stride, const int32_t* idx, const int32_t* n_sel,
                                float* out, const hg_host_desc* d) {
    if (!desc_ok(d) || !full || !idx || !n_sel || !out || full_stride < 1) return HG_ERR_INVALID_ARG;
    const int K = d->max_selected, G = d->num_q_heads / d->num_kv_heads;
    const float ninf = -std::numeric_limits<float>::infinity();
    parallel_for((int64_t)d->batch * d->num_q_heads, d->threads, [&](int64_t row) {
        const int b = (int)(row / d->num_q_heads), h = (int)(row % d->num_q_heads);
        const int nsel = std::max(0, std::min(n_sel[b], K));
        const int32_t* ix = idx + ((int64_t)b * d->num_kv_heads + h / G) * K;
        const float* src = full + row * full_stride;
        float* o = out + row * K;
        for (int i = 0; i < nsel; ++i) o[i] = (ix[i] >= 0 && ix[i] < full_stride) ? src[ix[i]] : ninf;
        for (int i = nsel; i < K; ++i) o[i] = ninf;
    });
    return HG_OK;
}

int32_t hg_host_select_positions(int32_t n_tokens, int32_t sinks, int32_t window, int32_t k, int32_t* idx_out) {
    if (!idx_out || n_tokens <= 0 || k <= 0) return 0;
    sinks = std::max(0, std::min(sinks, n_tokens));
    window = std::max(0, std::min(window, n_tokens - sinks));
    const int ns = std::min(sinks, k), nw = std::min(window, k - ns);
    int32_t w = 0;
    for (int i = 0; i < ns; ++i) idx_out[w++] = i;
    for (int i = n_tokens - nw; i < n_tokens; ++i) idx_out[w++] = i;   // the most recent nw tokens
    return w;
}

hg_status hg_host_select_ranked(const int32_t* ranking, int32_t batch, int32_t num_kv_heads, int32_t r,
                                const int32_t* n_host, int32_t k, int32_t* idx_out, int32_t* n_out) {
    if (!ranking || !n_host || !idx_out || !n_out || batch < 1 || num_kv_heads < 1 || r < 0 || k < 1) return HG_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b) {
        int n = std::max(0, std::min(k, n_host[b]));
        for (int g = 0; g < num_kv_heads; ++g) {                // the shortest valid prefix among the heads
            const int32_t* row = ranking + ((int64_t)b * num_kv_heads + g) * r;
            int valid = 0;
            while (valid < r && valid < n && row[valid] >= 0 && row[valid] < n_host[b]) ++valid;
            n = std::min(n, valid);
        }
        for (int g = 0; g < num_kv_heads; ++g) {
            const int32_t* row = ranking + ((int64_t)b * num_kv_heads + g) * r;
            int32_t* o = idx_out + ((int64_t)b * num_kv_heads + g) * k;
            for (int i = 0; i < k; ++i) o[i] = i < n ? row[i] : -1;
        }
        n_out[b] = n;
    }
    return HG_OK;
}

hg_status hg_host_gather_rows(const void* rows, const int32_t* idx, const int32_t* n_sel, void* dst, const hg_host_desc* d) {
    if (!desc_ok(d) || !rows || !idx || !n_sel || !dst) return HG_ERR_INVALID_ARG;
    const int D = d->head_dim, K = d->max_selected;
    const uint16_t* src = static_cast<const uint16_t*>(rows);
    uint16_t* out = static_cast<uint16_t*>(dst);
    parallel_for((int64_t)d->batch * d->num_kv_heads, d->threads, [&](int64_t bg) {
        const int b = (int)(bg / d->num_kv_heads), g = (int)(bg % d->num_kv_heads);
        const int n = std::max(0, std::min(n_sel[b], K));
        const int32_t* ix = idx + bg * K;
        uint16_t* o = out + bg * (int64_t)K * D;
        const uint16_t* base = src + (int64_t)b * d->seq_stride + (int64_t)g * d->head_stride;
        for (int i = 0; i < n; ++i) {
            if (ix[i] >= 0 && (d->num_rows <= 0 || ix[i] < d->num_rows)) copy_row(o + (int64_t)i * D, base + (int64_t)ix[i] * d->tok_stride, (size_t)D * 2);
            else memset(o + (int64_t)i * D, 0, (size_t)D * 2);       // padding or out of range: nothing is read
        }
        if (n < K) memset(o + (int64_t)n * D, 0, (size_t)(K - n) * D * 2);
        rows_written();
    });
    return HG_OK;
}

// ---- tiered host memory ---------------------------------------------------------------------------------------

int32_t hg_host_tier_nodes(void) {
#if defined(__linux__)
    // /sys/devices/system/node/has_memory: a list like "0" or "0-1,3"
    FILE* f = fopen("/sys/devices/system/node/has_memory", "r");
    if (!f) return 1;
    int count = 0, a = 0, b = 0;
    char sep = 0;
    while (fscanf(f, "%d", &a) == 1) {
        b = a;
        if (fscanf(f, "%c", &sep) == 1 && sep == '-') { if (fscanf(f, "%d", &b) != 1) b = a; if (fscanf(f, "%c", &sep) != 1) sep = 0; }
        count += b - a + 1;
        if (sep != ',') break;
    }
    fclose(f);
    return count > 0 ? count : 1;
#else
    return 1;
#endif
}

static bool node_has_memory(int node) {
#if defined(__linux__)
    char path[64];
    snprintf(path, sizeof path, "/sys/devices/system/node/node%d/meminfo", node);
    FILE* f = fopen(path, "r");
    if (!f) return false;
    fclose(f);
    return true;
#else
    return node == 0;
#endif
}

hg_status hg_host_tier_alloc(size_t bytes, int32_t node, void** out) {
    if (!out || bytes == 0 || node < 0 || node >= 1024) return HG_ERR_INVALID_ARG;
    *out = nullptr;
    if (!node_has_memory(node)) return HG_ERR_INVALID_ARG;
#if defined(__linux__)
    void* p = mmap(nullptr, bytes, PROT_READ | PROT_WRITE, MAP_PRIVATE | MAP_ANONYMOUS, -1, 0);
    if (p == MAP_FAILED) return HG_ERR_UNSUPPORTED;
    unsigned long mask[16] = {0};                      // 1024 nodes
    mask[node / (8 * sizeof(unsigned long))] |= 1ul << (node % (8 * sizeof(unsigned long)));
    const long mpol_bind = 2;                          // MPOL_BIND: pages of this range come from the nodes in the mask only
    if (syscall(SYS_mbind, p, bytes, mpol_bind, mask, (unsigned long)(sizeof mask * 8), 0u) != 0) {
        munmap(p, bytes);
        return HG_ERR_UNSUPPORTED;
    }
    *out = p;
    return HG_OK;
#else
    return HG_ERR_UNSUPPORTED;
#endif
}

void hg_host_tier_free(void* ptr, size_t bytes) {
#if defined(__linux__)
    if (ptr && bytes) munmap(ptr, bytes);
#endif
}

int32_t hg_host_tier_node_of(const void* ptr) {
#if defined(__linux__)
    if (!ptr) return -1;
    void* page = reinterpret_cast<void*>(reinterpret_cast<uintptr_t>(ptr) & ~(uintptr_t)4095);
    int status = -1;
    // move_pages with no target nodes only reports where each page is
    if (syscall(SYS_move_pages, 0, 1ul, &page, nullptr, &status, 0) != 0) return -1;
    return status >= 0 ? status : -1;
#else
    return -1;
#endif
}

void hg_sched_init(hg_sched_state* st, int32_t k_min) {
    if (!st) return;
    st->k = k_min;
    st->strategy = HG_SCHED_POST_QK;
}

void hg_sched_update(hg_sched_state* st, double t_gpu, double t_cpu, double t_tx, int32_t k_min, int32_t k_max,
                     int32_t step) {
    if (!st) return;
    if (step < 1) step = 1;
    if (k_max < k_min) k_max = k_min;
    if (t_cpu + t_tx <= t_gpu) {                       // the CPU stage is hidden behind the GPU stage:
        st->k = std::min(k_max, st->k + step);         // more tokens, in either selection mode
    } else if (st->k > k_min) {
        st->k = std::max(k_min, st->k - step);
    } else {
        st->strategy = HG_SCHED_PRE_QK;
    }
}

}  // extern "C"
