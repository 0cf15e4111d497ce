// Host-side companions declared in include/hybridgen_host.h: logits calculator, token selection, row
// gather and the feedback scheduler policy.  No CUDA here.
#include "hybridgen_host.h"

#include <math.h>
#include <string.h>

#include <algorithm>
#include <atomic>
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

float dot_scalar(const uint16_t* a, const uint16_t* b, int D, bool bf16) {
    float acc = 0.f;
    if (bf16) for (int d = 0; d < D; ++d) acc = fmaf(bf16_bits_to_float(a[d]), bf16_bits_to_float(b[d]), acc);
    else for (int d = 0; d < D; ++d) acc = fmaf(half_bits_to_float(a[d]), half_bits_to_float(b[d]), acc);
    return acc;
}

#if defined(__x86_64__)
__attribute__((target("avx2,fma,f16c"))) float dot_avx2(const uint16_t* a, const uint16_t* b, int D, bool bf16) {
    __m256 acc = _mm256_setzero_ps();
    for (int d = 0; d < D; d += 8) {
        const __m128i ra = _mm_loadu_si128(reinterpret_cast<const __m128i*>(a + d));
        const __m128i rb = _mm_loadu_si128(reinterpret_cast<const __m128i*>(b + d));
        __m256 fa, fb;
        if (bf16) {
            fa = _mm256_castsi256_ps(_mm256_slli_epi32(_mm256_cvtepu16_epi32(ra), 16));
            fb = _mm256_castsi256_ps(_mm256_slli_epi32(_mm256_cvtepu16_epi32(rb), 16));
        } else {
            fa = _mm256_cvtph_ps(ra);
            fb = _mm256_cvtph_ps(rb);
        }
        acc = _mm256_fmadd_ps(fa, fb, acc);
    }
    __m128 s = _mm_add_ps(_mm256_castps256_ps128(acc), _mm256_extractf128_ps(acc, 1));
    s = _mm_add_ps(s, _mm_movehl_ps(s, s));
    s = _mm_add_ss(s, _mm_shuffle_ps(s, s, 1));
    return _mm_cvtss_f32(s);
}
bool have_avx2() {
    static const bool ok = __builtin_cpu_supports("avx2") && __builtin_cpu_supports("fma") && __builtin_cpu_supports("f16c");
    return ok;
}
#endif

inline float dot16(const uint16_t* a, const uint16_t* b, int D, bool bf16) {
#if defined(__x86_64__)
    if (have_avx2()) return dot_avx2(a, b, D, bf16);
#endif
    return dot_scalar(a, b, D, bf16);
}

bool desc_ok(const hg_host_desc* d) {
    return d && d->struct_size >= sizeof(hg_host_desc) && d->batch >= 1 && d->num_kv_heads >= 1 && d->num_q_heads >= 1 &&
           d->num_q_heads % d->num_kv_heads == 0 && d->head_dim >= 8 && d->head_dim % 8 == 0 &&
           (d->dtype == HG_DTYPE_F16 || d->dtype == HG_DTYPE_BF16) && d->max_selected >= 1 && d->scale >= 0.f &&
           d->threads >= 0;
}

// Runs fn(i) for i in [0, n) on `threads` workers (0: one per core).
template <class F>
void parallel_for(int64_t n, int threads, F fn) {
    int nt = threads > 0 ? threads : (int)std::thread::hardware_concurrency();
    if (nt < 1) nt = 1;
    if ((int64_t)nt > n) nt = (int)n;
    if (nt <= 1) { for (int64_t i = 0; i < n; ++i) fn(i); return; }
    std::atomic<int64_t> next{0};
    std::vector<std::thread> pool;
    auto work = [&] { for (int64_t i; (i = next.fetch_add(1)) < n;) fn(i); };
    for (int t = 1; t < nt; ++t) pool.emplace_back(work);
    work();
    for (auto& t : pool) t.join();
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
    parallel_for((int64_t)d->batch * d->num_q_heads, d->threads, [&](int64_t row) {
        const int b = (int)(row / d->num_q_heads), h = (int)(row % d->num_q_heads), g = h / G;
        const int n = std::max(0, std::min(n_sel[b], K));
        const uint16_t* qrow = qp + row * D;
        const uint16_t* kb = kp + (int64_t)b * d->seq_stride + (int64_t)g * d->head_stride;
        const int32_t* ix = idx ? idx + ((int64_t)b * d->num_kv_heads + g) * K : nullptr;
        float* out = logits + row * K;
        for (int i = 0; i < n; ++i) {
            const int64_t t = ix ? ix[i] : i;
            out[i] = scale * dot16(qrow, kb + t * d->tok_stride, D, bf16);
        }
        for (int i = n; i < K; ++i) out[i] = -std::numeric_limits<float>::infinity();
    });
    return HG_OK;
}

hg_status hg_host_select_topk(const float* scores, int64_t rows, int64_t stride, const int32_t* n, int32_t k,
                              int32_t* idx_out, int32_t* n_out) {
    if (!scores || !n || !idx_out || rows < 0 || stride < 1 || k < 1) return HG_ERR_INVALID_ARG;
    parallel_for(rows, 0, [&](int64_t r) {
        const float* s = scores + r * stride;
        const int nv = (int)std::max<int64_t>(0, std::min<int64_t>(n[r], stride));
        std::vector<int32_t> cand;
        cand.reserve(nv);
        for (int i = 0; i < nv; ++i) if (!(s[i] != s[i])) cand.push_back(i);      // NaN is never selected
        const int take = std::min<int>(k, (int)cand.size());
        auto better = [&](int32_t a, int32_t b) { return s[a] > s[b] || (s[a] == s[b] && a < b); };
        if (take < (int)cand.size()) std::nth_element(cand.begin(), cand.begin() + take, cand.end(), better);
        cand.resize(take);
        std::sort(cand.begin(), cand.end());
        int32_t* out = idx_out + r * k;
        for (int i = 0; i < take; ++i) out[i] = cand[i];
        for (int i = take; i < k; ++i) out[i] = -1;
        if (n_out) n_out[r] = take;
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
        for (int i = 0; i < n; ++i) memcpy(o + (int64_t)i * D, base + (int64_t)ix[i] * d->tok_stride, (size_t)D * 2);
        if (n < K) memset(o + (int64_t)n * D, 0, (size_t)(K - n) * D * 2);
    });
    return HG_OK;
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
    if (t_cpu + t_tx <= t_gpu) {                       // the CPU stage is hidden behind the GPU stage
        if (st->strategy == HG_SCHED_PRE_QK) st->strategy = HG_SCHED_POST_QK;
        else st->k = std::min(k_max, st->k + step);
    } else if (st->k > k_min) {
        st->k = std::max(k_min, st->k - step);
    } else {
        st->strategy = HG_SCHED_PRE_QK;
    }
}

}  // extern "C"
