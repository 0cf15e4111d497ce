/*
 * fp64 CPU oracle for hybrid (token-split) decode attention.  TEST INFRASTRUCTURE ONLY:
 * tests, the smoke check and the bench's cpu_baseline leg may call it; the product never does.
 * It shares no code with the CUDA library.
 *
 * What it computes, for one query vector q (one sequence, one query head) against the K and V
 * rows of that head's KV head, over a set T of token positions:
 *
 *   logits      s_t = (sum_d q_d * K[t][d]) / sqrt(D)           (Section 2.1: Q x K^T / sqrt(d),
 *                                                                d = per-head dimension)
 *   FULL(T)     softmax over T of s, then the weighted sum of V rows (Section 2.1; Section 4.2,
 *               "conventional attention": logits, softmax over all tokens, value aggregation)
 *   PARTIAL(T)  (m, l, o) = (max_T s, sum_T e^{s_t-m}, sum_T e^{s_t-m} V_t): the un-normalised
 *               pieces of FULL(T); empty T gives (-inf, 0, 0)
 *   MERGE       log-sum-exp combination of partials over disjoint token sets; by Section 4.2's
 *               exactness claim (outputs identical to monolithic execution) it must equal
 *               FULL of the union
 *   PARTIAL from logits  the same triple from host-computed logits and gathered V rows (the device side of
 *               the paper's hand-off)
 *   LITERAL     the paper's own hand-off (Section 4.2 / workflow steps 2-5): each device computes
 *               raw logits for its own tokens, the logits and V rows are concatenated and put
 *               back in original token order, one softmax, one value aggregation
 *
 * Inputs are raw 16-bit patterns (IEEE binary16 or bfloat16); the decoders below turn a pattern
 * into the exact real value it denotes.  All arithmetic is double precision, tokens in ascending
 * order, no blocking or reordering.  Parity pins: see tests/test_oracle_pins.py (brute force,
 * split invariance, closed forms, a hand-worked example).  No function here is unpinned.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define HGO_F16 0
#define HGO_BF16 1

/* ---- exact 16-bit decoders ------------------------------------------------------------- */

double hgo_decode_f16(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0) v = ldexp((double)f, -24);                 /* subnormal: f * 2^-24 */
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -v : v;
}

double hgo_decode_bf16(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 7) & 0xff;
    int f = h & 0x7f;
    double v;
    if (e == 0) v = ldexp((double)f, -133);                /* subnormal: f * 2^-7 * 2^-126 */
    else if (e == 255) v = f ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)f / 128.0, e - 127);
    return sign ? -v : v;
}

static double dec(uint16_t h, int dtype) { return dtype == HGO_BF16 ? hgo_decode_bf16(h) : hgo_decode_f16(h); }

void hgo_decode(const uint16_t* bits, int64_t n, int dtype, double* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = dec(bits[i], dtype);
}

/* token index of the i-th member of T: idx[i] if an index list is given, else t0 + i */
static int64_t tok(const int64_t* idx, int64_t t0, int64_t i) { return idx ? idx[i] : t0 + i; }

/* ---- logits (Section 2.1) --------------------------------------------------------------- */

/* s[i] = scale * <q, K[tok_i]> ; K row t starts at K + t * tok_stride (elements). scale <= 0 means 1/sqrt(D). */
void hgo_logits(const uint16_t* q, const uint16_t* K, int64_t tok_stride, int D, int dtype, double scale,
                const int64_t* idx, int64_t t0, int64_t n, double* s) {
    if (!(scale > 0.0)) scale = 1.0 / sqrt((double)D);
    for (int64_t i = 0; i < n; ++i) {
        const uint16_t* row = K + tok(idx, t0, i) * tok_stride;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += dec(q[d], dtype) * dec(row[d], dtype);
        s[i] = acc * scale;
    }
}

/* ---- PARTIAL ---------------------------------------------------------------------------- */

void hgo_partial(const uint16_t* q, const uint16_t* K, const uint16_t* V, int64_t tok_stride, int D, int dtype,
                 double scale, const int64_t* idx, int64_t t0, int64_t n, double* m_out, double* l_out, double* o) {
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    if (n <= 0) { *m_out = -INFINITY; *l_out = 0.0; return; }
    double* s = (double*)malloc(sizeof(double) * (size_t)n);
    hgo_logits(q, K, tok_stride, D, dtype, scale, idx, t0, n, s);
    double m = s[0];
    for (int64_t i = 1; i < n; ++i) if (s[i] > m) m = s[i];
    double l = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double p = exp(s[i] - m);
        const uint16_t* row = V + tok(idx, t0, i) * tok_stride;
        l += p;
        for (int d = 0; d < D; ++d) o[d] += p * dec(row[d], dtype);
    }
    free(s);
    *m_out = m; *l_out = l;
}

/* ---- PARTIAL from given logits: the device side of the paper's hand-off (Section 4.2, CPU-side support /
 *      workflow steps 2-5): the host ships the logits s_i of n selected tokens and their V rows
 *      Vsel[i] (row i at Vsel + i * row_stride); the result is the same (m, l, o) a PARTIAL over those
 *      tokens gives.  Logits of -inf mark unselected slots; all -inf (or n = 0) is the empty partial. */
void hgo_partial_from_logits(const double* s, const uint16_t* Vsel, int64_t row_stride, int D, int dtype, int64_t n,
                             double* m_out, double* l_out, double* o) {
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    double m = -INFINITY;
    for (int64_t i = 0; i < n; ++i) if (s[i] > m) m = s[i];
    if (m == -INFINITY) { *m_out = -INFINITY; *l_out = 0.0; return; }
    double l = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        if (s[i] == -INFINITY) continue;
        double p = exp(s[i] - m);
        l += p;
        for (int d = 0; d < D; ++d) o[d] += p * dec(Vsel[i * row_stride + d], dtype);
    }
    *m_out = m; *l_out = l;
}

/* ---- FULL: softmax(q K^T / sqrt(D)) V and its log-sum-exp --------------------------------- */

void hgo_full(const uint16_t* q, const uint16_t* K, const uint16_t* V, int64_t tok_stride, int D, int dtype,
              double scale, const int64_t* idx, int64_t t0, int64_t n, double* out, double* lse) {
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (n <= 0) { *lse = -INFINITY; return; }
    double* s = (double*)malloc(sizeof(double) * (size_t)n);
    hgo_logits(q, K, tok_stride, D, dtype, scale, idx, t0, n, s);
    double M = s[0];
    for (int64_t i = 1; i < n; ++i) if (s[i] > M) M = s[i];
    double Z = 0.0;
    for (int64_t i = 0; i < n; ++i) Z += exp(s[i] - M);
    for (int64_t i = 0; i < n; ++i) {
        double w = exp(s[i] - M) / Z;                       /* softmax weight of token i */
        const uint16_t* row = V + tok(idx, t0, i) * tok_stride;
        for (int d = 0; d < D; ++d) out[d] += w * dec(row[d], dtype);
    }
    free(s);
    *lse = M + log(Z);
}

/* ---- MERGE ------------------------------------------------------------------------------ */

/* o is [n_src][D]. Sources with m = -inf are skipped; if all are, out = 0 and lse = -inf. */
void hgo_merge(int64_t n_src, const double* m, const double* l, const double* o, int D, double* out, double* lse) {
    double M = -INFINITY;
    for (int64_t i = 0; i < n_src; ++i) if (m[i] > M) M = m[i];
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (M == -INFINITY) { *lse = -INFINITY; return; }
    double L = 0.0;
    for (int64_t i = 0; i < n_src; ++i) {
        if (m[i] == -INFINITY) continue;
        double w = exp(m[i] - M);
        L += w * l[i];
        for (int d = 0; d < D; ++d) out[d] += w * o[i * (int64_t)D + d];
    }
    for (int d = 0; d < D; ++d) out[d] /= L;
    *lse = M + log(L);
}

/* ---- LITERAL: logits from two devices, concatenated in token order, one softmax ------------ */

typedef struct { int64_t t; double s; } hgo_pair;
static int cmp_pair(const void* a, const void* b) {
    int64_t x = ((const hgo_pair*)a)->t, y = ((const hgo_pair*)b)->t;
    return (x > y) - (x < y);
}

void hgo_literal(const uint16_t* q, const uint16_t* K, const uint16_t* V, int64_t tok_stride, int D, int dtype,
                 double scale, const int64_t* idx_a, int64_t n_a, const int64_t* idx_b, int64_t n_b,
                 double* out, double* lse) {
    int64_t n = n_a + n_b;
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (n <= 0) { *lse = -INFINITY; return; }
    double* sa = (double*)malloc(sizeof(double) * (size_t)(n_a > 0 ? n_a : 1));
    double* sb = (double*)malloc(sizeof(double) * (size_t)(n_b > 0 ? n_b : 1));
    hgo_logits(q, K, tok_stride, D, dtype, scale, idx_a, 0, n_a, sa);   /* device A's logit vector */
    hgo_logits(q, K, tok_stride, D, dtype, scale, idx_b, 0, n_b, sb);   /* device B's logit vector */
    hgo_pair* cat = (hgo_pair*)malloc(sizeof(hgo_pair) * (size_t)n);
    for (int64_t i = 0; i < n_a; ++i) { cat[i].t = idx_a[i]; cat[i].s = sa[i]; }
    for (int64_t i = 0; i < n_b; ++i) { cat[n_a + i].t = idx_b[i]; cat[n_a + i].s = sb[i]; }
    qsort(cat, (size_t)n, sizeof(hgo_pair), cmp_pair);                  /* original token order */
    double M = cat[0].s;
    for (int64_t i = 1; i < n; ++i) if (cat[i].s > M) M = cat[i].s;
    double Z = 0.0;
    for (int64_t i = 0; i < n; ++i) Z += exp(cat[i].s - M);
    for (int64_t i = 0; i < n; ++i) {
        double w = exp(cat[i].s - M) / Z;
        const uint16_t* row = V + cat[i].t * tok_stride;                /* the matching V row */
        for (int d = 0; d < D; ++d) out[d] += w * dec(row[d], dtype);
    }
    free(sa); free(sb); free(cat);
    *lse = M + log(Z);
}

/* ---- batched forms over a logical cache [B][Lmax][Hkv][D], threaded over (sequence, query head) --- */

typedef struct {
    const uint16_t *q, *K, *V;
    int B, Hq, Hkv, D, dtype;
    int64_t Lmax;
    double scale;
    const int64_t *range_lo, *range_hi;   /* per sequence: tokens [lo, hi) */
    int64_t chunk;                         /* chunk size (absolute grid), 0 = one piece */
    int64_t NC;                            /* chunk slots per (b,h) in the outputs */
    double *m, *l, *o;                     /* partial outputs [B][Hq][NC], [B][Hq][NC][D] */
    double *out, *lse;                     /* full outputs [B][Hq][D], [B][Hq] (mode 1) */
    int mode;                              /* 0 = chunked partials, 1 = FULL over [lo, hi) */
    int next;                              /* work counter */
    pthread_mutex_t mu;
} hgo_job;

static void run_item(hgo_job* J, int item) {
    int b = item / J->Hq, h = item % J->Hq;
    int g = h / (J->Hq / J->Hkv);                                   /* consecutive grouping of query heads */
    int64_t tok_stride = (int64_t)J->Hkv * J->D;
    const uint16_t* q = J->q + ((int64_t)b * J->Hq + h) * J->D;
    const uint16_t* K = J->K + ((int64_t)b * J->Lmax * J->Hkv + g) * J->D;
    const uint16_t* V = J->V + ((int64_t)b * J->Lmax * J->Hkv + g) * J->D;
    int64_t lo = J->range_lo[b], hi = J->range_hi[b];
    if (J->mode == 1) {
        hgo_full(q, K, V, tok_stride, J->D, J->dtype, J->scale, NULL, lo, hi > lo ? hi - lo : 0,
                 J->out + (int64_t)item * J->D, J->lse + item);
        return;
    }
    int64_t C = J->chunk > 0 ? J->chunk : (hi > lo ? hi - lo : 1);
    int64_t first = J->chunk > 0 ? lo / C : 0;
    for (int64_t c = 0; c < J->NC; ++c) {
        int64_t a, e;
        if (J->chunk > 0) { a = (first + c) * C; e = a + C; } else { a = c == 0 ? lo : hi; e = hi; }
        if (a < lo) a = lo;
        if (e > hi) e = hi;
        int64_t n = e > a ? e - a : 0;
        int64_t slot = (int64_t)item * J->NC + c;
        hgo_partial(q, K, V, tok_stride, J->D, J->dtype, J->scale, NULL, a, n, J->m + slot, J->l + slot,
                    J->o + slot * J->D);
    }
}

static void* worker(void* arg) {
    hgo_job* J = (hgo_job*)arg;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        int item = J->next++;
        pthread_mutex_unlock(&J->mu);
        if (item >= J->B * J->Hq) break;
        run_item(J, item);
    }
    return NULL;
}

static void run_job(hgo_job* J, int threads) {
    if (threads < 1) threads = 1;
    if (threads > 256) threads = 256;
    J->next = 0;
    pthread_mutex_init(&J->mu, NULL);
    pthread_t th[256];
    for (int i = 1; i < threads; ++i) pthread_create(&th[i], NULL, worker, J);
    worker(J);
    for (int i = 1; i < threads; ++i) pthread_join(th[i], NULL);
    pthread_mutex_destroy(&J->mu);
}

/* PARTIAL for every (b, h, chunk c): chunk c of sequence b covers absolute tokens
 * [(floor(lo_b/chunk)+c)*chunk, +chunk) clipped to [lo_b, hi_b); slots past the last chunk are empty. */
void hgo_chunked_partials(const uint16_t* q, const uint16_t* K, const uint16_t* V, int B, int Hq, int Hkv, int D,
                          int dtype, int64_t Lmax, double scale, const int64_t* lo, const int64_t* hi,
                          int64_t chunk, int64_t NC, double* m, double* l, double* o, int threads) {
    hgo_job J;
    memset(&J, 0, sizeof J);
    J.q = q; J.K = K; J.V = V; J.B = B; J.Hq = Hq; J.Hkv = Hkv; J.D = D; J.dtype = dtype; J.Lmax = Lmax;
    J.scale = scale; J.range_lo = lo; J.range_hi = hi; J.chunk = chunk; J.NC = NC; J.m = m; J.l = l; J.o = o;
    J.mode = 0;
    run_job(&J, threads);
}

/* FULL over [lo_b, hi_b) for every (b, h). */
void hgo_full_batch(const uint16_t* q, const uint16_t* K, const uint16_t* V, int B, int Hq, int Hkv, int D,
                    int dtype, int64_t Lmax, double scale, const int64_t* lo, const int64_t* hi,
                    double* out, double* lse, int threads) {
    hgo_job J;
    memset(&J, 0, sizeof J);
    J.q = q; J.K = K; J.V = V; J.B = B; J.Hq = Hq; J.Hkv = Hkv; J.D = D; J.dtype = dtype; J.Lmax = Lmax;
    J.scale = scale; J.range_lo = lo; J.range_hi = hi; J.out = out; J.lse = lse; J.mode = 1;
    run_job(&J, threads);
}
