/*
 * sla_oracle.c -- fp64 CPU oracle for N=2 Superlinear attention (span-search + span-attention).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, step-by-step restatement of
 * what the paper defines, used only by the tests, the smoke check and the benchmark's CPU-baseline
 * leg.  It shares no code, header, table or helper with the CUDA library and neither includes the
 * other.  The product path never calls it.
 *
 * What it follows (paper sections / equations / algorithm):
 *   - Anchor schedule, Section "Span attention" and the caption of the structural non-exclusion
 *     figure: for exponent p = 1/2 the anchors of query i sit at  t_s = i - (s+1)^2 + 1,
 *     s = 0, 1, 2, ...  (i, i-3, i-8, i-15, ...).
 *   - Search score, Section "Span search", first equation:  s_{i,t} = <Q_s(i), K_a(t)>,  K_a = K.
 *   - Top-k, Section "Span search", second equation, and Algorithm 1 step "TopK".
 *   - Span construction, Algorithm 1:  S_t = [max(0, t - b*l(i)), min(i, t + f*l(i))] (closed),
 *     l(i) = ceil(sqrt(i)) unless a fixed base length is given.
 *   - Span attention, Section "Span attention", equation for A_{i,t}: scaled dot-product softmax
 *     attention over the tokens of a span.
 *   - Combination, Section "Combination", both equations: alpha = softmax over the selected search
 *     scores, O_i = sum_t alpha_t A_{i,t}.
 *   - Sliding window W and DedupConcat, Algorithm 1 lines for W, T = Anchors(i) \ W and J_t.
 *
 * Readings taken where the paper is silent or inconsistent (all are conventions):
 *   R1  every anchor with t_s >= 0 is a candidate, i.e. (s+1)^2 <= i+1, n(i) = floor(sqrt(i+1));
 *   R2  spans are the closed interval of Algorithm 1 (so (b+f)*l + 1 tokens when unclipped);
 *   R3  l(i) is the exact integer ceiling of sqrt(i); l(0) = 0;
 *   R4  ties in top-k are broken towards the smaller stride index s (the nearer anchor) and the
 *       selected anchors are reported in (score descending, s ascending) order;
 *   R5  with fewer than k candidates all of them are taken and the tail is padded with
 *       anchor = -1, score = -infinity;
 *   R6  with grouped-query attention every query head routes on its own, scoring against the key
 *       head of its group (kv head = q head / (Hq / Hkv));
 *   R7  two output modes.  UNION: one softmax over the de-duplicated union of the selected spans
 *       (and the window) -- this reduces to dense causal attention when the selection covers every
 *       key.  PER_SPAN: Algorithm 1 literally -- one softmax per span (J_t = S_t united with W),
 *       then the gate of the Combination section.
 *   R8  the window W = [max(0, i-w+1), i] removes exactly the anchors with (s+1)^2 <= w;
 *   R9  for exponents other than 1/2 the anchor offset (s+1)^(1/p) and the base length i^p are real
 *       numbers; both are rounded UP to the next integer, after one part in 1e12 has been taken off
 *       so that a power that is an integer in exact arithmetic stays that integer (see ceil_pow).
 *
 * Parity pins (tests/test_oracle_*.py): the paper's worked example (i = 30), the anchor gap
 * sequence, the w = 1088 window adjacency, the closed-form work count and its L^{3/2} growth, the
 * coverage invariant (b >= 2), equality with textbook dense causal attention when top_k takes all
 * anchors, exhaustive scoring on tiny L, and the algebraic special cases.  Unpinned conventions
 * ("parity unpinned"): R1 versus the text's looser bound, R2's closed end-points, R4's tie order.
 *
 * Arithmetic is fp64 throughout; inputs are the fp32 / bf16 values the GPU reads, widened exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SLA_ORACLE_F32 0
#define SLA_ORACLE_BF16 1
#define SLA_ORACLE_F64 2

#define SLA_ORACLE_UNION 0
#define SLA_ORACLE_PER_SPAN 1

/* ------------------------------------------------------------------ integer helpers */

/* floor(sqrt(x)) for x >= 0, by integer search only (no floating point). */
int64_t sla_oracle_isqrt(int64_t x) {
    if (x <= 0) return 0;
    int64_t r = 0;
    while ((r + 1) * (r + 1) <= x) r++;
    return r;
}

/* fast variant used inside the row loops; corrected to the exact integer result. */
static int64_t isqrt_fast(int64_t x) {
    if (x <= 0) return 0;
    int64_t r = (int64_t)floor(sqrt((double)x));
    while (r * r > x) r--;
    while ((r + 1) * (r + 1) <= x) r++;
    return r;
}

/* smallest r with r*r >= x  (reading R3: l(i) = ceil(sqrt(i)) as an integer). */
int64_t sla_oracle_ceil_isqrt(int64_t x) {
    if (x <= 0) return 0;
    int64_t r = isqrt_fast(x);
    if (r * r < x) r++;
    return r;
}

/*
 * General exponents (Section "Span attention": anchors at i - (s+1)^(1/p) + 1 for general p; Section
 * "Training": search_exponent for the stride pattern, span_exponent for the span length).  The paper
 * does not say how the real number (s+1)^(1/p) becomes a position; the reading taken here (R9 above): it is rounded UP to
 * an integer, after taking off one part in 1e12 so that a power that is an integer in exact
 * arithmetic (p = 1/3: cubes) is not pushed to the next one by the rounding of 1/p and pow (their
 * relative error is a few 1e-15; positions stay below 2^31, so the margin is far below 1).  For
 * p = 1/2 the offsets are the exact squares, computed in integers.
 */
static int64_t ceil_pow(double base, double expo) {
    double x = pow(base, expo);
    return (int64_t)ceil(x - 1e-12 * x);
}

/* Distance of the stride-s anchor from position i + 1: o_s = ceil((s+1)^(1/p)). */
int64_t sla_oracle_stride_offset(int64_t s, double p) {
    if (p == 0.5) return (s + 1) * (s + 1);
    return ceil_pow((double)(s + 1), 1.0 / p);
}

/* Number of strides whose anchor exists for query position i: o_s <= i + 1 (reading R1). */
int64_t sla_oracle_n_strides(int64_t i, double p) {
    int64_t n = 0;
    while (sla_oracle_stride_offset(n, p) <= i + 1) n++;
    return n;
}

/* Base span length l(i): the fixed value when span_len > 0, else the paper's rule ceil(i^p_span)
 * (an exact integer ceil-sqrt for p_span = 1/2). */
int64_t sla_oracle_base_len(int64_t i, int64_t span_len, double p_span) {
    if (span_len > 0) return span_len;
    if (i <= 0) return 0;
    if (p_span == 0.5) return sla_oracle_ceil_isqrt(i);
    return ceil_pow((double)i, p_span);
}

/*
 * Candidate anchors of query position i (Algorithm 1: T = Anchors(i) \ W).
 * Writes the key positions in stride order (s ascending, i.e. nearest first) and, when s_out is not
 * NULL, the stride index of each.  Returns how many there are; writes at most cap of them.
 */
int64_t sla_oracle_anchors(int64_t i, int64_t window, double p, int64_t *t_out, int64_t *s_out, int64_t cap) {
    int64_t n = 0;
    int64_t w_lo = window > 0 ? (i - window + 1 > 0 ? i - window + 1 : 0) : i + 1; /* W = [w_lo, i] */
    for (int64_t s = 0;; s++) {
        int64_t t = i - sla_oracle_stride_offset(s, p) + 1;
        if (t < 0) break;                      /* reading R1 */
        if (window > 0 && t >= w_lo) continue; /* anchor lies inside W: not a candidate */
        if (n < cap) {
            if (t_out) t_out[n] = t;
            if (s_out) s_out[n] = s;
        }
        n++;
    }
    return n;
}

/* Closed span S_t of Algorithm 1. */
void sla_oracle_span(int64_t i, int64_t t, int64_t ell, int64_t b, int64_t f, int64_t *lo,
                     int64_t *hi) {
    int64_t a = t - b * ell;
    int64_t z = t + f * ell;
    *lo = a > 0 ? a : 0;
    *hi = z < i ? z : i;
}

/* ------------------------------------------------------------------ element access */

static inline double load_elem(const void *base, int dtype, int64_t idx) {
    if (dtype == SLA_ORACLE_F32) return (double)((const float *)base)[idx];
    if (dtype == SLA_ORACLE_F64) return ((const double *)base)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16; /* bf16 -> fp32, exact */
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static double dot_row(const void *a, int64_t a_off, const void *b, int64_t b_off, int dtype, int D) {
    double acc = 0.0;
    for (int d = 0; d < D; d++) acc += load_elem(a, dtype, a_off + d) * load_elem(b, dtype, b_off + d);
    return acc;
}

int sla_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ span search */

/*
 * Span-search for the query rows of one call.
 *
 * q_s : [B, Hq, Lq, D]   routing queries; row r is query position q_pos0 + r
 * k   : [B, Hkv, kv_cap, D]   keys, positions 0 .. Lkv-1 valid
 * rows: optional list of n_rows row offsets in [0, Lq) to evaluate (NULL = all Lq rows, R = Lq);
 *       outputs are indexed [B, Hq, R, ...] in the order of that list.
 * out_anchor [B,Hq,R,top_k] int32 key positions (score descending, then s ascending; -1 padding)
 * out_score  [B,Hq,R,top_k] fp64 (search_scale * dot; -inf padding)
 * out_gap    [B,Hq,R] fp64, score of the k-th selected minus score of the best rejected candidate
 *            (+inf when nothing was rejected); may be NULL
 * n_dots     number of score dot products evaluated (work count); may be NULL
 * returns 0, or -1 on a bad argument.
 */
int sla_oracle_span_search(const void *q_s, const void *k, int dtype, int B, int Hq, int Hkv, int D,
                           int64_t Lq, int64_t q_pos0, int64_t Lkv, int64_t kv_cap, int top_k,
                           int64_t window, double search_scale, double search_exponent,
                           const int64_t *rows, int64_t n_rows, int32_t *out_anchor, double *out_score,
                           double *out_gap, int64_t *n_dots) {
    if (!q_s || !k || B <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv || D <= 0 || Lq <= 0 || top_k <= 0 ||
        q_pos0 < 0 || q_pos0 + Lq > Lkv || Lkv > kv_cap || window < 0 || !(search_exponent > 0.0) ||
        !(search_exponent < 1.0))
        return -1;
    const int G = Hq / Hkv;
    const int64_t R = rows ? n_rows : Lq;
    int64_t dots_total = 0;
    int bad = 0;

#pragma omp parallel for collapse(2) schedule(dynamic, 16) reduction(+ : dots_total)
    for (int64_t bh = 0; bh < (int64_t)B * Hq; bh++) {
        for (int64_t rr = 0; rr < R; rr++) {
            const int b = (int)(bh / Hq), h = (int)(bh % Hq), g = h / G;
            const int64_t r = rows ? rows[rr] : rr;
            if (r < 0 || r >= Lq) { bad = 1; continue; }
            const int64_t i = q_pos0 + r;
            const int64_t n_all = search_exponent == 0.5 ? isqrt_fast(i + 1)
                                                         : sla_oracle_n_strides(i, search_exponent); /* strides with t >= 0 */
            double *sc = (double *)malloc(sizeof(double) * (size_t)(n_all > 0 ? n_all : 1));
            int64_t *tt = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_all > 0 ? n_all : 1));
            char *taken = (char *)calloc((size_t)(n_all > 0 ? n_all : 1), 1);
            const int64_t n = sla_oracle_anchors(i, window, search_exponent, tt, NULL, n_all);
            const int64_t q_off = (((int64_t)b * Hq + h) * Lq + r) * D;
            for (int64_t c = 0; c < n; c++) {
                const int64_t k_off = (((int64_t)b * Hkv + g) * kv_cap + tt[c]) * D;
                sc[c] = search_scale * dot_row(q_s, q_off, k, k_off, dtype, D);
            }
            dots_total += n;
            /* top-k by repeated arg-max; candidates are stored in stride order, so the strict
               '>' keeps the smaller stride on ties (reading R4). */
            const int64_t o = (((int64_t)b * Hq + h) * R + rr) * top_k;
            for (int j = 0; j < top_k; j++) {
                int64_t best = -1;
                for (int64_t c = 0; c < n; c++)
                    if (!taken[c] && (best < 0 || sc[c] > sc[best])) best = c;
                if (best < 0) {
                    out_anchor[o + j] = -1;
                    out_score[o + j] = -INFINITY;
                } else {
                    taken[best] = 1;
                    out_anchor[o + j] = (int32_t)tt[best];
                    out_score[o + j] = sc[best];
                }
            }
            if (out_gap) {
                double rej = -INFINITY;
                for (int64_t c = 0; c < n; c++)
                    if (!taken[c] && sc[c] > rej) rej = sc[c];
                double kth = out_score[o + top_k - 1];
                out_gap[((int64_t)b * Hq + h) * R + rr] =
                    (rej == -INFINITY || kth == -INFINITY) ? INFINITY : kth - rej;
            }
            free(sc); free(tt); free(taken);
        }
    }
    if (n_dots) *n_dots = dots_total;
    return bad ? -1 : 0;
}

/* ------------------------------------------------------------------ span attention */

typedef struct { int64_t lo, hi; } interval_t;

static int cmp_interval(const void *a, const void *b) {
    const interval_t *x = (const interval_t *)a, *y = (const interval_t *)b;
    if (x->lo != y->lo) return x->lo < y->lo ? -1 : 1;
    if (x->hi != y->hi) return x->hi < y->hi ? -1 : 1;
    return 0;
}

/*
 * Softmax attention of one query row over the de-duplicated union of n closed intervals
 * (DedupConcat of Algorithm 1).  Two plain passes: maximum, then normalised sum.
 * Writes out[D] and returns lse = log sum_j exp(x_j); an empty set gives out = 0, lse = -inf.
 * *pairs is incremented by the number of (query, key) pairs visited.
 */
static double attend_union(const void *q, int64_t q_off, const void *k, const void *v, int64_t kv_off,
                           int dtype, int D, double scale, interval_t *iv, int n, double *out,
                           int64_t *pairs) {
    for (int d = 0; d < D; d++) out[d] = 0.0;
    qsort(iv, (size_t)n, sizeof(interval_t), cmp_interval);
    /* pass 1: maximum logit over the distinct positions */
    double mx = -INFINITY;
    int64_t next_free = 0, cnt = 0;
    for (int a = 0; a < n; a++) {
        int64_t j0 = iv[a].lo > next_free ? iv[a].lo : next_free;
        for (int64_t j = j0; j <= iv[a].hi; j++) {
            double x = scale * dot_row(q, q_off, k, kv_off + j * D, dtype, D);
            if (x > mx) mx = x;
            cnt++;
        }
        if (iv[a].hi + 1 > next_free) next_free = iv[a].hi + 1;
    }
    *pairs += cnt;
    if (cnt == 0) return -INFINITY;
    /* pass 2: sum of exponentials and the weighted value sum */
    double den = 0.0;
    next_free = 0;
    for (int a = 0; a < n; a++) {
        int64_t j0 = iv[a].lo > next_free ? iv[a].lo : next_free;
        for (int64_t j = j0; j <= iv[a].hi; j++) {
            double x = scale * dot_row(q, q_off, k, kv_off + j * D, dtype, D);
            double e = exp(x - mx);
            den += e;
            for (int d = 0; d < D; d++) out[d] += e * load_elem(v, dtype, kv_off + j * D + d);
        }
        if (iv[a].hi + 1 > next_free) next_free = iv[a].hi + 1;
    }
    for (int d = 0; d < D; d++) out[d] /= den;
    return mx + log(den);
}

/*
 * Span-attention for the query rows of one call.
 *
 * q      : [B, Hq, Lq, D]; k, v : [B, Hkv, kv_cap, D]
 * anchor : [B, Hq, R, top_k] int32 key positions, -1 = none
 * score  : [B, Hq, R, top_k] fp64 search scores (PER_SPAN gate only; may be NULL in UNION mode)
 * out    : [B, Hq, R, D] fp64
 * lse    : [B, Hq, R] fp64.  UNION: log-sum-exp of the logits over the attended set.  PER_SPAN: a
 *          single value is not defined for a gated mixture, so lse holds the value of the first
 *          (best-scoring) selected span and lse_span, if not NULL, [B,Hq,R,top_k] holds each
 *          span's own value (-inf for padding).
 * n_pairs: number of (query, key) pairs attended (work count); may be NULL
 */
int sla_oracle_span_attention(const void *q, const void *k, const void *v, int dtype, int B, int Hq,
                              int Hkv, int D, int64_t Lq, int64_t q_pos0, int64_t Lkv,
                              int64_t kv_cap, int top_k, int64_t span_len, int64_t back_factor,
                              int64_t fwd_factor, int64_t window, int mode, double softmax_scale,
                              double span_exponent, const int64_t *rows, int64_t n_rows, const int32_t *anchor,
                              const double *score, double *out, double *lse, double *lse_span,
                              int64_t *n_pairs) {
    if (!q || !k || !v || !anchor || B <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv || D <= 0 || Lq <= 0 ||
        top_k <= 0 || q_pos0 < 0 || q_pos0 + Lq > Lkv || Lkv > kv_cap || window < 0 ||
        back_factor < 0 || fwd_factor < 0 || (mode == SLA_ORACLE_PER_SPAN && !score))
        return -1;
    const int G = Hq / Hkv;
    const int64_t R = rows ? n_rows : Lq;
    int64_t pairs_total = 0;
    int bad = 0;

#pragma omp parallel for collapse(2) schedule(dynamic, 4) reduction(+ : pairs_total)
    for (int64_t bh = 0; bh < (int64_t)B * Hq; bh++) {
        for (int64_t rr = 0; rr < R; rr++) {
            const int b = (int)(bh / Hq), h = (int)(bh % Hq), g = h / G;
            const int64_t r = rows ? rows[rr] : rr;
            if (r < 0 || r >= Lq) { bad = 1; continue; }
            const int64_t i = q_pos0 + r;
            const int64_t ell = sla_oracle_base_len(i, span_len, span_exponent);
            const int64_t q_off = (((int64_t)b * Hq + h) * Lq + r) * D;
            const int64_t kv_off = ((int64_t)b * Hkv + g) * kv_cap * D;
            const int64_t row = ((int64_t)b * Hq + h) * R + rr;
            const int32_t *an = anchor + row * top_k;
            double *o = out + row * D;
            interval_t *iv = (interval_t *)malloc(sizeof(interval_t) * (size_t)(top_k + 1));
            interval_t win;
            win.lo = i - window + 1 > 0 ? i - window + 1 : 0;
            win.hi = i;
            int64_t pairs = 0;

            if (mode == SLA_ORACLE_UNION) {
                int n = 0;
                for (int j = 0; j < top_k; j++) {
                    if (an[j] < 0) continue;
                    if (an[j] > i) { bad = 1; continue; }
                    sla_oracle_span(i, an[j], ell, back_factor, fwd_factor, &iv[n].lo, &iv[n].hi);
                    n++;
                }
                if (window > 0) iv[n++] = win;
                lse[row] = attend_union(q, q_off, k, v, kv_off, dtype, D, softmax_scale, iv, n, o, &pairs);
            } else {
                /* Algorithm 1: A_t per span over J_t = S_t + W, then the softmax gate. */
                double *a_t = (double *)malloc(sizeof(double) * (size_t)D);
                double smax = -INFINITY, sden = 0.0;
                int n_sel = 0;
                for (int j = 0; j < top_k; j++)
                    if (an[j] >= 0) { n_sel++; if (score[row * top_k + j] > smax) smax = score[row * top_k + j]; }
                for (int d = 0; d < D; d++) o[d] = 0.0;
                lse[row] = -INFINITY;
                if (n_sel == 0) {
                    /* Algorithm 1, empty selection: attention over the window alone. */
                    if (window > 0) {
                        iv[0] = win;
                        lse[row] = attend_union(q, q_off, k, v, kv_off, dtype, D, softmax_scale, iv, 1, o, &pairs);
                    }
                    for (int j = 0; j < top_k && lse_span; j++) lse_span[row * top_k + j] = -INFINITY;
                } else {
                    for (int j = 0; j < top_k; j++)
                        if (an[j] >= 0) sden += exp(score[row * top_k + j] - smax);
                    int first = 1;
                    for (int j = 0; j < top_k; j++) {
                        if (an[j] < 0) { if (lse_span) lse_span[row * top_k + j] = -INFINITY; continue; }
                        if (an[j] > i) { bad = 1; continue; }
                        int n = 0;
                        sla_oracle_span(i, an[j], ell, back_factor, fwd_factor, &iv[n].lo, &iv[n].hi);
                        n++;
                        if (window > 0) iv[n++] = win;
                        double l_t = attend_union(q, q_off, k, v, kv_off, dtype, D, softmax_scale, iv, n, a_t, &pairs);
                        double alpha = exp(score[row * top_k + j] - smax) / sden;
                        for (int d = 0; d < D; d++) o[d] += alpha * a_t[d];
                        if (lse_span) lse_span[row * top_k + j] = l_t;
                        if (first) { lse[row] = l_t; first = 0; }
                    }
                }
                free(a_t);
            }
            pairs_total += pairs;
            free(iv);
        }
    }
    if (n_pairs) *n_pairs = pairs_total;
    return bad ? -1 : 0;
}

/* ------------------------------------------------------------------ decode step */

/*
 * One decode step: the single query at position i = n_ctx - 1 against a cache that already holds
 * the current token (Section "Kernel design", decoding path).  It is the prefill definition with
 * Lq = 1 and q_pos0 = n_ctx - 1, composed from the two routines above.
 *
 * q_s, q : [B, Hq, D];  k_cache, v_cache : [B, Hkv, kv_cap, D]
 * outputs: out [B,Hq,D], lse [B,Hq], out_anchor/out_score [B,Hq,top_k], out_gap [B,Hq] (nullable)
 */
int sla_oracle_decode_step(const void *q_s, const void *q, const void *k_cache, const void *v_cache,
                           int dtype, int B, int Hq, int Hkv, int D, int64_t n_ctx, int64_t kv_cap,
                           int top_k, int64_t span_len, int64_t back_factor, int64_t fwd_factor,
                           int64_t window, int mode, double search_scale, double softmax_scale,
                           double search_exponent, double span_exponent,
                           int32_t *out_anchor, double *out_score, double *out_gap, double *out,
                           double *lse, int64_t *n_dots, int64_t *n_pairs) {
    if (n_ctx <= 0) return -1;
    int rc = sla_oracle_span_search(q_s, k_cache, dtype, B, Hq, Hkv, D, 1, n_ctx - 1, n_ctx, kv_cap,
                                    top_k, window, search_scale, search_exponent, NULL, 0, out_anchor,
                                    out_score, out_gap, n_dots);
    if (rc) return rc;
    return sla_oracle_span_attention(q, k_cache, v_cache, dtype, B, Hq, Hkv, D, 1, n_ctx - 1, n_ctx,
                                     kv_cap, top_k, span_len, back_factor, fwd_factor, window, mode,
                                     softmax_scale, span_exponent, NULL, 0, out_anchor, out_score, out, lse,
                                     NULL, n_pairs);
}
