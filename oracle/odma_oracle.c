/*
 * CPU checker for slab-KV decode attention and the ODMA bucket allocator.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * GPU library must compute.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it; the library never does, and the two share no code.
 *
 * Part 1 - attention.  Dense softmax attention in fp64, two passes, no chunking,
 *   no running rescale.  The paper reuses its serving stack's stock decode kernel
 *   (Section IV-A) and never writes the formula; it is the textbook one:
 *   s_j = q.k_j / sqrt(D), p = softmax(s), o = sum_j p_j v_j, with query head h
 *   reading KV head h div (Hq/Hkv).
 *   Pins: fp64 library attention, closed forms, invariants, a high-precision
 *   evaluation on tiny inputs (tests/test_oracle_attention.py).
 *   K and V may also be held as E4M3 codes with a dequantisation scale per layer (an
 *   8-bit slab): the format is written out from its definition, rounding is a search for
 *   the nearest code.  Pins: the format's published special values, an independent
 *   library's widening of all 256 codes and its rounding on 200,000 numbers and every
 *   midpoint, attention over the dequantised values (tests/test_oracle_e4m3.py).
 *
 * Part 2 - allocator.  One owner entry per token of the pool; every placement is
 *   found by scanning that array.  Steps follow Section III (B: uncertainty
 *   inflation and routing, C: quantile boundaries from a sliding window, Eq. 2,
 *   D: Large Bucket with pre-emptive routing and allocate-and-copy migration,
 *   E: reserve/release) and Section IV-C (new boundaries apply to newly admitted
 *   requests only).  Where the paper is silent the reading taken is written at
 *   the step.
 *   Pins: a hand-computed placement table, numpy's nearest-rank quantile, exact
 *   rational arithmetic for the inflation, structural invariants
 *   (tests/test_oracle_allocator.py).
 *   Adaptive recalibration under drift has no worked example in the paper:
 *   parity unpinned against the paper for that part (pinned to the library
 *   quantile only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* Part 1: attention                                                          */
/* ------------------------------------------------------------------------- */

enum { ORA_F32 = 0, ORA_BF16 = 1, ORA_E4M3 = 2 };

/*
 * The 8-bit floating-point format E4M3 (OCP 8-bit floating point specification, the "fn"
 * variant: no infinities): bit 7 sign, bits 6..3 exponent E (bias 7), bits 2..0 mantissa M.
 *   E = 0:            value = M * 2^-9                (subnormal; M = 0 is zero)
 *   E = 15 and M = 7: NaN
 *   otherwise:        value = (1 + M/8) * 2^(E - 7)   (largest: E = 15, M = 6: 448)
 */
static double e4m3_value(uint8_t code) {
    int e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    v = e == 0 ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, e - 7);
    return (code & 0x80) ? -v : v;
}

/*
 * Nearest E4M3 code of an fp32 number by the definition of rounding.  The magnitudes of
 * codes 0x00..0x7E increase with the code, so the nearest finite value is one of the two
 * that enclose |y|: lo = the largest code whose value is <= |y| (found by bisection) and
 * lo + 1.  Distances are exact in fp64; of two equally close values the one with the even
 * code (round to nearest even: neighbours are consecutive codes); anything beyond +-448
 * saturates to +-448.  NaN gives the NaN code.
 */
static uint8_t e4m3_nearest(float y) {
    double a = fabs((double)y);
    uint8_t sign = signbit(y) ? 0x80 : 0;
    int lo = 0, hi = 0x7E, best;
    if (isnan(y)) return (uint8_t)(sign | 0x7F);
    if (a >= e4m3_value(0x7E)) return (uint8_t)(sign | 0x7E);
    while (hi - lo > 1) {               /* invariant: value(lo) <= a < value(hi) */
        int mid = (lo + hi) / 2;
        if (e4m3_value((uint8_t)mid) <= a) lo = mid; else hi = mid;
    }
    {
        double d_lo = a - e4m3_value((uint8_t)lo), d_hi = e4m3_value((uint8_t)hi) - a;
        if (d_lo < d_hi) best = lo;
        else if (d_hi < d_lo) best = hi;
        else best = (lo & 1) == 0 ? lo : hi;
    }
    return (uint8_t)(sign | best);
}

/* Widen one stored element to fp64.  bf16 is the upper half of an fp32. */
static double widen(const void* p, size_t i, int dtype) {
    if (dtype == ORA_F32) return (double)((const float*)p)[i];
    if (dtype == ORA_E4M3) return e4m3_value(((const uint8_t*)p)[i]);
    uint32_t bits = (uint32_t)((const uint16_t*)p)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

void oracle_e4m3_widen(const uint8_t* codes, size_t n, double* out) {
    for (size_t i = 0; i < n; ++i) out[i] = e4m3_value(codes[i]);
}

void oracle_e4m3_round(const float* x, size_t n, uint8_t* codes) {
    for (size_t i = 0; i < n; ++i) codes[i] = e4m3_nearest(x[i]);
}

/*
 * What an append into an E4M3 slab stores: the row's elements (fp32 or bf16, as given)
 * widened to fp32, multiplied IN FP32 by inv_scale (the caller's fp32 reciprocal of the
 * dequantisation scale; one rounding, the precision the GPU path takes the same decision
 * in), rounded to the nearest code.
 */
void oracle_e4m3_quantize(const void* x, int dtype, size_t n, float inv_scale, uint8_t* codes) {
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
    for (long long i = 0; i < (long long)n; ++i) {
        volatile float y = (float)widen(x, (size_t)i, dtype) * inv_scale;
        codes[i] = e4m3_nearest(y);
    }
}

/*
 * One (request, query head).  q: [Hq][D] of type qdtype.  K, V: [L][Hkv][D] of type kvdtype,
 * token-major (the checker's own store; it never sees the device layout); a stored key
 * element stands for widen(K) * k_scale, a value element for widen(V) * v_scale (both 1 for
 * fp32 and bf16 stores; the per-layer dequantisation scales of an E4M3 store).  out: [D].
 * weights (may be NULL): [L] softmax weights.  Returns the log-sum-exp of the scaled scores.
 */
static double attention_head(const void* q, int qdtype, const void* K, const void* V, int kvdtype,
                             double k_scale, double v_scale, int L, int h, int Hq, int Hkv, int D,
                             double* out, double* weights) {
    int group = Hq / Hkv;
    int kappa = h / group;
    double* s = (double*)malloc(sizeof(double) * (size_t)L);
    double mx = -INFINITY;
    for (int j = 0; j < L; ++j) {
        double dot = 0.0;
        for (int d = 0; d < D; ++d)
            dot += widen(q, (size_t)h * D + d, qdtype) *
                   (widen(K, ((size_t)j * Hkv + kappa) * D + d, kvdtype) * k_scale);
        s[j] = dot / sqrt((double)D);
        if (s[j] > mx) mx = s[j];
    }
    double sum = 0.0;
    for (int j = 0; j < L; ++j) sum += exp(s[j] - mx);
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int j = 0; j < L; ++j) {
        double p = exp(s[j] - mx) / sum;
        if (weights) weights[j] = p;
        for (int d = 0; d < D; ++d)
            out[d] += p * (widen(V, ((size_t)j * Hkv + kappa) * D + d, kvdtype) * v_scale);
    }
    free(s);
    return mx + log(sum);
}

/*
 * A batch of n requests.  q: [n][Hq][D]; K[i], V[i]: [L[i]][Hkv][D];
 * out: [n][Hq][D] fp64; lse: [n][Hq] fp64 or NULL.  Work is spread over
 * (request, head) pairs; returns the number of threads used.
 */
static int attention_batch(int n, const void* q, int qdtype, const void* const* K, const void* const* V,
                           int kvdtype, double k_scale, double v_scale, const int32_t* L, int Hq, int Hkv,
                           int D, double* out, double* lse, int threads) {
    size_t esz = qdtype == ORA_F32 ? 4 : 2;
    int used = 1;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#pragma omp parallel
    {
#pragma omp single
        used = omp_get_num_threads();
    }
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int w = 0; w < n * Hq; ++w) {
        int i = w / Hq, h = w % Hq;
        const char* qi = (const char*)q + (size_t)i * Hq * D * esz;
        double l = attention_head(qi, qdtype, K[i], V[i], kvdtype, k_scale, v_scale, L[i], h, Hq, Hkv, D,
                                  out + ((size_t)i * Hq + h) * D, NULL);
        if (lse) lse[(size_t)i * Hq + h] = l;
    }
    return used;
}

int oracle_decode_attention(int n, const void* q, const void* const* K, const void* const* V,
                            const int32_t* L, int Hq, int Hkv, int D, int dtype, double* out,
                            double* lse, int threads) {
    return attention_batch(n, q, dtype, K, V, dtype, 1.0, 1.0, L, Hq, Hkv, D, out, lse, threads);
}

/* The same with K and V held as E4M3 codes (one byte per element) and their scales. */
int oracle_decode_attention_e4m3(int n, const void* q, int qdtype, const void* const* K,
                                 const void* const* V, float k_scale, float v_scale, const int32_t* L,
                                 int Hq, int Hkv, int D, double* out, double* lse, int threads) {
    return attention_batch(n, q, qdtype, K, V, ORA_E4M3, (double)k_scale, (double)v_scale, L, Hq, Hkv, D,
                           out, lse, threads);
}

/* Softmax weights of one (request, head), for the invariants tests. */
double oracle_attention_weights(const void* q, const void* K, const void* V, int L, int h, int Hq,
                                int Hkv, int D, int dtype, double* out, double* weights) {
    return attention_head(q, dtype, K, V, dtype, 1.0, 1.0, L, h, Hq, Hkv, D, out, weights);
}

/*
 * The split-then-merge identity the GPU path relies on, in fp64: attention over
 * [0,L) computed as independent pieces [c0,c1), each giving (m, l, o), merged by
 * M = max m, l = sum l_s e^{m_s-M}, o = sum o_s e^{m_s-M} / l.  Used by a test to
 * show the merge formula equals the dense result; not used as the checker itself.
 */
void oracle_attention_chunked(const void* q, const void* K, const void* V, int L, int h, int Hq,
                              int Hkv, int D, int dtype, int chunk, double* out) {
    int group = Hq / Hkv, kappa = h / group;
    int pieces = (L + chunk - 1) / chunk;
    double* m = (double*)malloc(sizeof(double) * pieces);
    double* l = (double*)malloc(sizeof(double) * pieces);
    double* o = (double*)calloc((size_t)pieces * D, sizeof(double));
    for (int c = 0; c < pieces; ++c) {
        int j0 = c * chunk, j1 = j0 + chunk < L ? j0 + chunk : L;
        double* s = (double*)malloc(sizeof(double) * (j1 - j0));
        m[c] = -INFINITY;
        for (int j = j0; j < j1; ++j) {
            double dot = 0.0;
            for (int d = 0; d < D; ++d)
                dot += widen(q, (size_t)h * D + d, dtype) *
                       widen(K, ((size_t)j * Hkv + kappa) * D + d, dtype);
            s[j - j0] = dot / sqrt((double)D);
            if (s[j - j0] > m[c]) m[c] = s[j - j0];
        }
        l[c] = 0.0;
        for (int j = j0; j < j1; ++j) {
            double e = exp(s[j - j0] - m[c]);
            l[c] += e;
            for (int d = 0; d < D; ++d)
                o[(size_t)c * D + d] += e * widen(V, ((size_t)j * Hkv + kappa) * D + d, dtype);
        }
        free(s);
    }
    double M = -INFINITY, lsum = 0.0;
    for (int c = 0; c < pieces; ++c)
        if (m[c] > M) M = m[c];
    for (int c = 0; c < pieces; ++c) lsum += l[c] * exp(m[c] - M);
    for (int d = 0; d < D; ++d) {
        double acc = 0.0;
        for (int c = 0; c < pieces; ++c) acc += o[(size_t)c * D + d] * exp(m[c] - M);
        out[d] = acc / lsum;
    }
    free(m);
    free(l);
    free(o);
}

/* ------------------------------------------------------------------------- */
/* Part 2: allocator                                                          */
/* ------------------------------------------------------------------------- */

/* Status codes: the numeric values are part of the library's documented interface. */
enum {
    ORA_OK = 0,
    ORA_ERR_INVALID = 1,
    ORA_ERR_NOMEM = 2,
    ORA_ERR_UNKNOWN_REQ = 3,
    ORA_ERR_DUP_REQ = 4,
    ORA_ERR_OVERFLOW = 5
};

#define ORA_MAX_BUCKETS 8

typedef struct {
    uint64_t id;
    int64_t base, cap, len;
    int pool;   /* 0 main, 1 Large Bucket (safety pool) */
    int bucket; /* index of the boundary used, -1 for the Large Bucket */
    int migrations;
    int live;
} ora_req;

typedef struct {
    /* pool carving, in tokens */
    int64_t T, S, M, G, max_len;
    int32_t* own; /* own[t] = index into reqs of the owner of token t, -1 when free */
    /* requests (append-only table, linear search) */
    ora_req* reqs;
    int64_t n_reqs, cap_reqs;
    /* Adaptive Bucket Manager (Section III-C) */
    int n_buckets;                       /* boundaries in force */
    int64_t bounds[ORA_MAX_BUCKETS];
    int n_levels;                        /* B quantile levels p_i = p_num[i] / p_den */
    int64_t p_num[ORA_MAX_BUCKETS], p_den;
    int64_t W, R;
    int64_t* window; /* realised lengths, oldest first */
    int64_t n_window;
    int64_t observed;
    uint64_t epoch;
    /* uncertainty policy (Section III-B): gamma, tau in thousandths */
    int64_t gamma_pm, tau_pm;
    int64_t growth;
    int large_fixed;
    /* counters */
    int64_t completed, sum_len_completed, sum_cap_completed, migrations, nomem, routed_large;
    int64_t safety_peak;
} ora_alloc;

static int64_t ceil_g(int64_t x, int64_t G) { return (x + G - 1) / G * G; }
static int64_t floor_g(int64_t x, int64_t G) { return x / G * G; }

/*
 * Carve the pool.  The paper gives no units; reading: everything is counted in
 * tokens, one token = layers * 2 * kv_heads * head_dim * elem_bytes bytes, sizes are
 * rounded down to the granule G, and the Large Bucket takes an integer percentage.
 */
ora_alloc* ora_create(uint64_t bytes, int layers, int kv_heads, int head_dim, int elem_bytes,
                      int safety_pct, int64_t max_len, int64_t G, int64_t W, int64_t R,
                      int n_buckets, const int32_t* p_num, int32_t p_den, int gamma_pm, int tau_pm,
                      int growth, int large_fixed) {
    if (G < 1 || max_len < G || max_len % G != 0 || n_buckets < 1 || n_buckets > ORA_MAX_BUCKETS ||
        W < 1 || R < 1 || p_den < 1)
        return NULL;
    ora_alloc* a = (ora_alloc*)calloc(1, sizeof *a);
    uint64_t per_tok = (uint64_t)layers * 2u * (uint64_t)kv_heads * (uint64_t)head_dim * (uint64_t)elem_bytes;
    a->G = G;
    a->T = floor_g((int64_t)(bytes / per_tok), G);
    a->S = floor_g(a->T * safety_pct / 100, G);
    a->M = a->T - a->S;
    a->max_len = max_len;
    a->own = (int32_t*)malloc(sizeof(int32_t) * (size_t)(a->T > 0 ? a->T : 1));
    for (int64_t t = 0; t < a->T; ++t) a->own[t] = -1;
    a->n_levels = n_buckets;
    for (int i = 0; i < n_buckets; ++i) a->p_num[i] = p_num[i];
    a->p_den = p_den;
    a->W = W;
    a->R = R;
    a->window = (int64_t*)malloc(sizeof(int64_t) * (size_t)W);
    a->gamma_pm = gamma_pm;
    a->tau_pm = tau_pm;
    a->growth = growth;
    a->large_fixed = large_fixed;
    /* until boundaries are set or learned there is a single bucket: max_len */
    a->n_buckets = 1;
    a->bounds[0] = max_len;
    return a;
}

void ora_destroy(ora_alloc* a) {
    if (!a) return;
    free(a->own);
    free(a->reqs);
    free(a->window);
    free(a);
}

void ora_geometry(const ora_alloc* a, int64_t* out3) {
    out3[0] = a->T;
    out3[1] = a->S;
    out3[2] = a->M;
}

/* Static / initial boundaries: strictly increasing multiples of G, at most max_len. */
int ora_set_buckets(ora_alloc* a, const int32_t* b, int n) {
    if (n < 1 || n > ORA_MAX_BUCKETS) return ORA_ERR_INVALID;
    for (int i = 0; i < n; ++i) {
        if (b[i] < 1 || b[i] % a->G != 0 || b[i] > a->max_len) return ORA_ERR_INVALID;
        if (i > 0 && b[i] <= b[i - 1]) return ORA_ERR_INVALID;
    }
    for (int i = 0; i < n; ++i) a->bounds[i] = b[i];
    a->n_buckets = n;
    a->epoch += 1;
    return ORA_OK;
}

int ora_get_buckets(const ora_alloc* a, int32_t* b, uint64_t* epoch) {
    for (int i = 0; i < a->n_buckets; ++i) b[i] = (int32_t)a->bounds[i];
    *epoch = a->epoch;
    return a->n_buckets;
}

static ora_req* find_live(ora_alloc* a, uint64_t id) {
    /* newest first: live requests are the recent ones */
    for (int64_t i = a->n_reqs - 1; i >= 0; --i)
        if (a->reqs[i].live && a->reqs[i].id == id) return &a->reqs[i];
    return NULL;
}

/*
 * Lowest-address placement: the smallest multiple of G in [lo, hi - cap] whose cap
 * tokens are all free.  "Per-size free lists" (Section III-E) are read as an index
 * over exactly this result.  Returns -1 when nothing fits.
 */
static int64_t first_fit(const ora_alloc* a, int64_t lo, int64_t hi, int64_t cap) {
    for (int64_t base = lo; base + cap <= hi; base += a->G) {
        int free_run = 1;
        for (int64_t t = base; t < base + cap; ++t)
            if (a->own[t] != -1) {
                free_run = 0;
                break;
            }
        if (free_run) return base;
    }
    return -1;
}

static ora_req* new_req(ora_alloc* a, uint64_t id) {
    if (a->n_reqs == a->cap_reqs) {
        a->cap_reqs = a->cap_reqs ? a->cap_reqs * 2 : 64;
        a->reqs = (ora_req*)realloc(a->reqs, sizeof(ora_req) * (size_t)a->cap_reqs);
    }
    ora_req* r = &a->reqs[a->n_reqs++];
    memset(r, 0, sizeof *r);
    r->id = id;
    r->live = 1;
    return r;
}

static void mark(ora_alloc* a, int64_t base, int64_t cap, int32_t who) {
    for (int64_t t = base; t < base + cap; ++t) a->own[t] = who;
}

static int64_t safety_in_use(const ora_alloc* a) {
    int64_t n = 0;
    for (int64_t t = a->M; t < a->T; ++t) n += a->own[t] != -1;
    return n;
}

/*
 * Large Bucket placement (Section III-D).  Reading: a slab of ceil_G(need) tokens,
 * capped at max_len (or always max_len when large_fixed), lowest address inside the
 * safety region [M, T).
 */
static int place_large(ora_alloc* a, int64_t need, int64_t* base, int64_t* cap) {
    int64_t c = a->large_fixed ? a->max_len : ceil_g(need, a->G);
    if (c > a->max_len) c = a->max_len;
    int64_t b = first_fit(a, a->M, a->T, c);
    if (b < 0) return ORA_ERR_NOMEM;
    *base = b;
    *cap = c;
    return ORA_OK;
}

static void fill_slab(const ora_req* r, uint64_t epoch, int64_t* out5) {
    out5[0] = r->base;
    out5[1] = r->cap;
    out5[2] = r->pool;
    out5[3] = r->bucket;
    out5[4] = (int64_t)epoch;
}

static int reserve_large(ora_alloc* a, uint64_t id, int64_t need, int64_t* out5) {
    int64_t base, cap;
    int rc = place_large(a, need, &base, &cap);
    if (rc != ORA_OK) {
        a->nomem += 1;
        return rc;
    }
    ora_req* r = new_req(a, id);
    r->base = base;
    r->cap = cap;
    r->pool = 1;
    r->bucket = -1;
    mark(a, base, cap, (int32_t)(r - a->reqs));
    a->routed_large += 1;
    int64_t u = safety_in_use(a);
    if (u > a->safety_peak) a->safety_peak = u;
    fill_slab(r, a->epoch, out5);
    return ORA_OK;
}

/*
 * reserve (Section III-E): P is the predicted TOTAL length (prompt + generation).
 * The bucket is the first boundary b_i >= P (a length equal to the boundary fits);
 * the slab takes b_i tokens at the lowest free address of the main region [0, M).
 * P beyond the last boundary goes to the Large Bucket.  A full main region is an
 * error for the caller's admission control; ordinary requests never spill into the
 * safety pool, which is budgeted for the tail.
 */
int ora_reserve(ora_alloc* a, uint64_t id, int64_t P, int64_t* out5) {
    if (P < 1) return ORA_ERR_INVALID;
    if (find_live(a, id)) return ORA_ERR_DUP_REQ;
    if (P > a->bounds[a->n_buckets - 1] || P > a->max_len)
        return reserve_large(a, id, P < a->max_len ? P : a->max_len, out5);
    int bi = 0;
    while (a->bounds[bi] < P) ++bi;
    int64_t cap = a->bounds[bi];
    int64_t base = first_fit(a, 0, a->M, cap);
    if (base < 0) {
        a->nomem += 1;
        return ORA_ERR_NOMEM;
    }
    ora_req* r = new_req(a, id);
    r->base = base;
    r->cap = cap;
    r->pool = 0;
    r->bucket = bi;
    mark(a, base, cap, (int32_t)(r - a->reqs));
    fill_slab(r, a->epoch, out5);
    return ORA_OK;
}

/*
 * Uncertainty-aware reserve (Section III-B): L' = L_hat (1 + gamma u), rounded up,
 * in integers with gamma and u in thousandths; u > tau goes straight to the Large
 * Bucket (pre-emptive routing, Section III-D).
 */
int ora_reserve_uncertain(ora_alloc* a, uint64_t id, int64_t L_hat, int64_t u_pm, int64_t* out5) {
    if (L_hat < 1 || u_pm < 0 || u_pm > 1000) return ORA_ERR_INVALID;
    int64_t inflated = (L_hat * (1000000 + a->gamma_pm * u_pm) + 999999) / 1000000;
    if (u_pm > a->tau_pm) {
        if (find_live(a, id)) return ORA_ERR_DUP_REQ;
        return reserve_large(a, id, inflated < a->max_len ? inflated : a->max_len, out5);
    }
    return ora_reserve(a, id, inflated, out5);
}

/*
 * Reactive migration (Sections III-D, IV-C): when the request needs more tokens
 * than its slab holds, a Large Bucket slab is allocated FIRST, the tokens are
 * copied, and only then is the old slab released.  Reading for the new size:
 * max(need, growth * current length), capped at max_len.
 */
int ora_ensure(ora_alloc* a, uint64_t id, int64_t need, int64_t* out5, int32_t* migrated) {
    ora_req* r = find_live(a, id);
    *migrated = 0;
    if (!r) return ORA_ERR_UNKNOWN_REQ;
    if (need <= r->cap) {
        fill_slab(r, a->epoch, out5);
        return ORA_OK;
    }
    if (need > a->max_len) return ORA_ERR_OVERFLOW;
    int64_t want = a->growth * r->len;
    if (want < need) want = need;
    if (want > a->max_len) want = a->max_len;
    int64_t base, cap;
    int rc = place_large(a, want, &base, &cap);
    if (rc != ORA_OK) {
        a->nomem += 1;
        return rc;
    }
    int32_t who = (int32_t)(r - a->reqs);
    mark(a, base, cap, who);        /* allocate ... */
    int64_t u = safety_in_use(a);   /* peak occupancy counts the moment both slabs are held */
    if (u > a->safety_peak) a->safety_peak = u;
    mark(a, r->base, r->cap, -1);   /* ... (copy) ... then release the old slab */
    r->base = base;
    r->cap = cap;
    r->pool = 1;
    r->bucket = -1;
    r->migrations += 1;
    a->migrations += 1;
    *migrated = 1;
    fill_slab(r, a->epoch, out5);
    return ORA_OK;
}

/* The request's KV length grew by n_new tokens (they must fit the slab). */
int ora_add_len(ora_alloc* a, uint64_t id, int64_t n_new) {
    ora_req* r = find_live(a, id);
    if (!r) return ORA_ERR_UNKNOWN_REQ;
    if (n_new < 0 || r->len + n_new > r->cap) return ORA_ERR_OVERFLOW;
    r->len += n_new;
    return ORA_OK;
}

int64_t ora_get_len(ora_alloc* a, uint64_t id) {
    ora_req* r = find_live(a, id);
    return r ? r->len : -1;
}

static int cmp_i64(const void* x, const void* y) {
    int64_t a = *(const int64_t*)x, b = *(const int64_t*)y;
    return (a > b) - (a < b);
}

/*
 * Eq. 2: b_i = Q_{p_i}(L) over the sliding window.  Reading: nearest-rank order
 * statistic x_(ceil(p n)) of the n values in the window, rounded up to the granule
 * and capped at max_len.  Equal boundaries may result; lookup takes the first.
 */
static void recalibrate(ora_alloc* a) {
    int64_t n = a->n_window;
    int64_t* sorted = (int64_t*)malloc(sizeof(int64_t) * (size_t)n);
    memcpy(sorted, a->window, sizeof(int64_t) * (size_t)n);
    qsort(sorted, (size_t)n, sizeof(int64_t), cmp_i64);
    a->n_buckets = a->n_levels;
    for (int i = 0; i < a->n_levels; ++i) {
        int64_t rank = (a->p_num[i] * n + a->p_den - 1) / a->p_den;
        if (rank < 1) rank = 1;
        if (rank > n) rank = n;
        int64_t b = ceil_g(sorted[rank - 1], a->G);
        if (b > a->max_len) b = a->max_len;
        a->bounds[i] = b;
    }
    free(sorted);
    a->epoch += 1;
}

/*
 * release (Section III-E) + logging of the realised length (Section III-A): the
 * slab's tokens become free, the realised total length enters the window (oldest
 * value leaves once W are held), and every R-th completion re-derives the
 * boundaries.  Live slabs keep their capacity (Section IV-C).
 */
int ora_release(ora_alloc* a, uint64_t id) {
    ora_req* r = find_live(a, id);
    if (!r) return ORA_ERR_UNKNOWN_REQ;
    mark(a, r->base, r->cap, -1);
    r->live = 0;
    a->completed += 1;
    a->sum_len_completed += r->len;
    a->sum_cap_completed += r->cap;
    if (a->n_window == a->W) {
        memmove(a->window, a->window + 1, sizeof(int64_t) * (size_t)(a->W - 1));
        a->n_window -= 1;
    }
    a->window[a->n_window++] = r->len;
    a->observed += 1;
    if (a->observed % a->R == 0) recalibrate(a);
    return ORA_OK;
}

/*
 * Counters.  Utilisation (Section V) = sum_len_completed / sum_cap_completed: the
 * actual KV use over the capacity the allocator had reserved for the request when
 * it completed.  out: live, reserved_live, used_live, completed, sum_len_completed,
 * sum_cap_completed, migrations, nomem, routed_large, safety_live, safety_peak,
 * observed.
 */
void ora_stats(const ora_alloc* a, int64_t* out12) {
    int64_t live = 0, reserved = 0, used = 0;
    for (int64_t i = 0; i < a->n_reqs; ++i)
        if (a->reqs[i].live) {
            live += 1;
            reserved += a->reqs[i].cap;
            used += a->reqs[i].len;
        }
    out12[0] = live;
    out12[1] = reserved;
    out12[2] = used;
    out12[3] = a->completed;
    out12[4] = a->sum_len_completed;
    out12[5] = a->sum_cap_completed;
    out12[6] = a->migrations;
    out12[7] = a->nomem;
    out12[8] = a->routed_large;
    out12[9] = safety_in_use(a);
    out12[10] = a->safety_peak;
    out12[11] = a->observed;
}

/* Raw owner array, for the no-overlap invariant test. */
const int32_t* ora_owner_array(const ora_alloc* a) { return a->own; }

/* Live requests: fills ids/base/cap/len/pool (each n_max long), returns the count. */
int64_t ora_live(const ora_alloc* a, int64_t n_max, uint64_t* ids, int64_t* base, int64_t* cap,
                 int64_t* len, int32_t* pool) {
    int64_t k = 0;
    for (int64_t i = 0; i < a->n_reqs && k < n_max; ++i)
        if (a->reqs[i].live) {
            ids[k] = a->reqs[i].id;
            base[k] = a->reqs[i].base;
            cap[k] = a->reqs[i].cap;
            len[k] = a->reqs[i].len;
            pool[k] = a->reqs[i].pool;
            ++k;
        }
    return k;
}
