/*
 * CPU oracle for one Adaptive Mass-Segmented (AMS) KV-compression event.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, sequential statement of
 * what the compression step computes, written from the paper's Section 3,
 * Eq. 1, Algorithm 1 and the two display equations of the paged-compaction
 * appendix.  It shares no code, header, table or constant with the CUDA path and
 * must never be linked or called by it.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may use it.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fPIC -shared   (never -ffast-math)
 *
 * Arithmetic convention ("canonical arithmetic").  The paper works in real
 * numbers; its prefix sums and threshold tests decide integers (cut positions,
 * quotas).  So that those integers have one right answer, every elementwise
 * floating-point operation below is one IEEE-754 round-to-nearest operation (no
 * fused multiply-add) and every sum over tokens that feeds a decision is a sum
 * of 64-bit integers obtained by fixed-point conversion with FIX_BITS = 36
 * fractional bits.  A normalisation x / total is evaluated as x * (1 / total),
 * the reciprocal rounded once per sequence.  Per token this departs from the real-valued definition by
 * less than 2^-36 of the total mass.
 *
 * Pins (see tests, CPU-only): Eq. 1 closed form and sum-to-one; cuts against an
 * exact rational brute force; uniform mass => equal segments; quotas summing to
 * the budget with their bounds; one segment => library top-k; beta = 1 => EMA
 * off; lambda = 0 => credit equals mass; gather equals dense indexing; TOVA
 * with one query row => library softmax; KeyDiff => library cosine similarity;
 * usage smoothing => library zero-padded average pooling and a hand-computed case;
 * expected-attention logits => Monte-Carlo mean of exp(q.k/sqrt(D)) over sampled Gaussian
 * queries, zero covariance => the one-query TOVA softmax, isotropic covariance => closed form.
 * EMA weights (beta on the current mass, 1 - beta on the normalised credit) and
 * the must-keep order (suffix gives way before the sinks) against exact rationals
 * and hand-worked cases; quota rounding (halves up) and the visiting order of the
 * adjustment step against hand-worked cases; the reciprocal normalisation against
 * exact integer division.
 * Parity unpinned (invariants and hand-made examples of this reading only, the
 * paper fixes neither): merge direction and the order of merge vs split; the
 * choice of "roughly equal" split sizes; the padding value of the causal
 * observation window when W > 1; for the expected-attention score, the order
 * softmax -> group mean -> (+ eps) -> value norm (the paper prints no formula; the
 * Gaussian closed form itself is pinned to its definition).
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define FIX_BITS 36

typedef struct {
    int32_t n_segments; /* S: thresholds k/S, i.e. target segment mass 1/S      */
    int32_t l_min;      /* segments shorter than this are merged                 */
    int32_t l_max;      /* segments longer than this are split; 0 = never split  */
    int32_t q_min;      /* guaranteed quota per segment                          */
    int32_t n_sink;     /* must-keep prefix                                      */
    int32_t n_last;     /* must-keep suffix                                      */
    float ema_lambda;   /* credit decay                                          */
    float ema_beta;     /* mixing weight of the current mass; 1 = credit unused  */
    float eps;          /* Eq. 1 epsilon                                         */
    int32_t fixed_segments; /* ablation "fixed-length segments": cuts at k T / S   */
    int32_t uniform_quotas; /* ablation "w/o mass-weighted quotas": share by length */
} orc_params;

/* ------------------------------------------------------------------------- */
/* bf16 and the paged layout                                                 */
/* ------------------------------------------------------------------------- */

static double bf16_to_double(uint16_t b)
{
    uint32_t w = (uint32_t)b << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* Physical layout: pages[layer][page][slot][kv_head][d], bf16, slot < page_size.
 * The block table row maps logical position p to page table[p / page_size]; the
 * row is shared by all layers and KV heads (paged-compaction appendix). */
typedef struct {
    const uint16_t *pages;
    int64_t num_pages;
    int32_t page_size, n_kv_heads, head_dim;
} orc_pool;

static int64_t row_offset(const orc_pool *P, int layer, int32_t page, int slot, int h)
{
    return ((((int64_t)layer * P->num_pages + page) * P->page_size + slot) * P->n_kv_heads + h) *
           (int64_t)P->head_dim;
}

static const uint16_t *k_row(const orc_pool *P, int layer, const int32_t *table_row, int t, int h)
{
    return P->pages + row_offset(P, layer, table_row[t / P->page_size], t % P->page_size, h);
}

/* ------------------------------------------------------------------------- */
/* Scorers                                                                    */
/* ------------------------------------------------------------------------- */

/* TOVA-style observation-window usage (Section 3.2; Algorithm 1 step 1; the
 * "mass construction" paragraph of the implementation appendix).
 * Rows r = (query head g of the GQA group, window query j), G*W of them; q holds
 * them as [G][W][D].  Window query j sits at position T-W+j, so with `causal` it
 * sees tokens t <= T-W+j.  Each row is a softmax of q.k/sqrt(D) over the tokens
 * it sees.  A (row, token) pair the row cannot see is filled with the largest
 * probability seen anywhere in the window; the usage of a token is the mean over
 * all rows. */
int orc_score_tova(const uint16_t *pages, int64_t num_pages, int32_t page_size, int32_t n_kv_heads,
                   int32_t head_dim, int32_t layer, int32_t h, const int32_t *table_row, int32_t T,
                   const uint16_t *q, int32_t G, int32_t W, int32_t causal, float *u_out)
{
    orc_pool P = {pages, num_pages, page_size, n_kv_heads, head_dim};
    const int rows = G * W;
    if (T < 1 || rows < 1 || W > T) return -1;
    double *p = (double *)malloc(sizeof(double) * (size_t)rows * (size_t)T);
    int32_t *last_valid = (int32_t *)malloc(sizeof(int32_t) * (size_t)rows);
    if (!p || !last_valid) { free(p); free(last_valid); return -2; }
    const double scale = 1.0 / sqrt((double)head_dim);
    double p_max = 0.0;
    for (int r = 0; r < rows; ++r) {
        const int j = r % W;
        const int lv = causal ? (T - W + j) : (T - 1);
        last_valid[r] = lv;
        const uint16_t *qr = q + (int64_t)r * head_dim;
        double *pr = p + (int64_t)r * T;
        double mx = -INFINITY;
        for (int t = 0; t <= lv; ++t) {
            const uint16_t *kt = k_row(&P, layer, table_row, t, h);
            double acc = 0.0;
            for (int d = 0; d < head_dim; ++d) acc += bf16_to_double(qr[d]) * bf16_to_double(kt[d]);
            pr[t] = acc * scale;
            if (pr[t] > mx) mx = pr[t];
        }
        double Z = 0.0;
        for (int t = 0; t <= lv; ++t) { pr[t] = exp(pr[t] - mx); Z += pr[t]; }
        for (int t = 0; t <= lv; ++t) { pr[t] /= Z; if (pr[t] > p_max) p_max = pr[t]; }
    }
    for (int t = 0; t < T; ++t) {
        double a = 0.0;
        for (int r = 0; r < rows; ++r) a += (t <= last_valid[r]) ? p[(int64_t)r * T + t] : p_max;
        u_out[t] = (float)(a / (double)rows);
    }
    free(p);
    free(last_valid);
    return 0;
}

/* KeyDiff-style key-only score: negative cosine similarity between a key and the
 * mean key of its (sequence, KV head) cache, so keys unlike the average rank
 * high (baseline table of the paper; the benchmark configuration fixes the
 * anchor as the per-head mean key). */
int orc_score_keydiff(const uint16_t *pages, int64_t num_pages, int32_t page_size,
                      int32_t n_kv_heads, int32_t head_dim, int32_t layer, int32_t h,
                      const int32_t *table_row, int32_t T, float *g_out)
{
    orc_pool P = {pages, num_pages, page_size, n_kv_heads, head_dim};
    if (T < 1) return -1;
    double *mu = (double *)calloc((size_t)head_dim, sizeof(double));
    if (!mu) return -2;
    for (int t = 0; t < T; ++t) {
        const uint16_t *kt = k_row(&P, layer, table_row, t, h);
        for (int d = 0; d < head_dim; ++d) mu[d] += bf16_to_double(kt[d]);
    }
    double mu2 = 0.0;
    for (int d = 0; d < head_dim; ++d) { mu[d] /= (double)T; mu2 += mu[d] * mu[d]; }
    const double mu_norm = sqrt(mu2);
    for (int t = 0; t < T; ++t) {
        const uint16_t *kt = k_row(&P, layer, table_row, t, h);
        double dot = 0.0, k2 = 0.0;
        for (int d = 0; d < head_dim; ++d) {
            const double kd = bf16_to_double(kt[d]);
            dot += kd * mu[d];
            k2 += kd * kd;
        }
        double den = sqrt(k2) * mu_norm;
        if (den < 1e-30) den = 1e-30;
        g_out[t] = (float)(-dot / den);
    }
    free(mu);
    return 0;
}

static const uint16_t *v_row(const orc_pool *P, int layer, const int32_t *table_row, int t, int h)
{
    return P->pages + row_offset(P, layer, table_row[t / P->page_size], t % P->page_size, h);
}

/* Expected-attention score (the scorer behind the paper's "AMS-Expected" rows; the
 * paper names it, its regularisation coefficient epsilon = 1e-2 and the work it comes
 * from, but prints no formula: what follows is a READING, the closed form that the
 * cited work's idea gives when the future queries of a head are modelled as Gaussian).
 * For a query q ~ N(mu, Sigma) the expected unnormalised attention weight of key k is
 * the Gaussian moment-generating function
 *     E[exp(q.k / sqrt(D))] = exp(mu.k / sqrt(D) + k^T Sigma k / (2 D)).
 * Per query head r of the KV head's GQA group: logit l_{r,t} = mu_r.k_t / sqrt(D) +
 * k_t^T Sigma_r k_t / (2 D), softmax over the T cached tokens, mean over the G heads of
 * the group, then (a_t + eps) * |v_t|_2 (the value norm weighs what a token would
 * contribute).  The query statistics are inputs (they come from the model's hidden
 * states, outside this step): mean fp32 [G][D], cov bf16 [G][D][D] (need not be
 * symmetric: only its symmetric part matters to the quadratic form). */
int orc_score_expected(const uint16_t *k_pages, const uint16_t *v_pages, int64_t num_pages, int32_t page_size,
                       int32_t n_kv_heads, int32_t head_dim, int32_t layer, int32_t h, const int32_t *table_row,
                       int32_t T, const float *mean, const uint16_t *cov, int32_t G, float eps, float *g_out)
{
    orc_pool PK = {k_pages, num_pages, page_size, n_kv_heads, head_dim};
    orc_pool PV = {v_pages, num_pages, page_size, n_kv_heads, head_dim};
    const int D = head_dim;
    if (T < 1 || G < 1) return -1;
    double *a = (double *)calloc((size_t)T, sizeof(double));
    double *l = (double *)malloc(sizeof(double) * (size_t)T);
    double *kd = (double *)malloc(sizeof(double) * (size_t)D);
    if (!a || !l || !kd) { free(a); free(l); free(kd); return -2; }
    for (int r = 0; r < G; ++r) {
        const float *mu = mean + (int64_t)r * D;
        const uint16_t *S = cov + (int64_t)r * D * D;
        double mx = -INFINITY;
        for (int t = 0; t < T; ++t) {
            const uint16_t *kt = k_row(&PK, layer, table_row, t, h);
            for (int j = 0; j < D; ++j) kd[j] = bf16_to_double(kt[j]);
            double lin = 0.0, quad = 0.0;
            for (int j = 0; j < D; ++j) {
                lin += (double)mu[j] * kd[j];
                double sk = 0.0; /* (Sigma k)_j */
                for (int i = 0; i < D; ++i) sk += bf16_to_double(S[(int64_t)j * D + i]) * kd[i];
                quad += kd[j] * sk;
            }
            l[t] = lin / sqrt((double)D) + quad / (2.0 * (double)D);
            if (l[t] > mx) mx = l[t];
        }
        double Z = 0.0;
        for (int t = 0; t < T; ++t) { l[t] = exp(l[t] - mx); Z += l[t]; }
        for (int t = 0; t < T; ++t) a[t] += l[t] / Z;
    }
    for (int t = 0; t < T; ++t) {
        const uint16_t *vt = v_row(&PV, layer, table_row, t, h);
        double v2 = 0.0;
        for (int j = 0; j < D; ++j) { const double x = bf16_to_double(vt[j]); v2 += x * x; }
        g_out[t] = (float)((a[t] / (double)G + (double)eps) * sqrt(v2));
    }
    free(a); free(l); free(kd);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Step 1: quality mass (Eq. 1)                                               */
/* ------------------------------------------------------------------------- */

/* w_t = max(u_t, 0) + eps in fp32 (NaN counts as 0, +inf as FLT_MAX), then the
 * fixed-point image A_t = floor(w_t * 2^(FIX_BITS - e)), e = exponent just above
 * the largest w, so A_t < 2^FIX_BITS and the sum stays below 2^53. */
void orc_fixed_point(const float *x, int32_t T, uint64_t *A, uint64_t *sum_out)
{
    float mx = 0.0f;
    for (int t = 0; t < T; ++t) if (x[t] > mx) mx = x[t];
    uint64_t s = 0;
    if (mx > 0.0f) {
        const int e = ilogbf(mx) + 1;
        for (int t = 0; t < T; ++t) {
            A[t] = (uint64_t)floor(ldexp((double)x[t], FIX_BITS - e));
            s += A[t];
        }
    } else {
        for (int t = 0; t < T; ++t) A[t] = 0;
    }
    *sum_out = s;
}

/* Optional smoothing of the usage scores along the sequence before Eq. 1 (Algorithm 1,
 * step 1: "optionally smooth"; the default configuration of the implementation-details
 * appendix names a small 1-D average pooling).  Window of k positions (k odd) centred on
 * t, positions outside [0, T) count as zero and the divisor is always k (the convention
 * of a zero-padded average pooling with stride 1).  The sum runs over the positions inside
 * the sequence from left to right in fp32, one rounding per addition, then one division:
 * a fixed order, so that the result has one value.  k = 1 leaves u as it is. */
void orc_smooth_usage(const float *u, int32_t T, int32_t k, float *out)
{
    const int r = k / 2;
    for (int t = 0; t < T; ++t) {
        if (k <= 1) { out[t] = u[t]; continue; }
        float s = 0.0f;
        const int lo = t - r < 0 ? 0 : t - r, hi = t + r > T - 1 ? T - 1 : t + r;
        for (int j = lo; j <= hi; ++j) s = s + u[j];
        out[t] = s / (float)k;
    }
}

void orc_weights(const float *u, int32_t T, float eps, float *w)
{
    for (int t = 0; t < T; ++t) {
        float v = fmaxf(u[t], 0.0f) + eps; /* fmaxf returns the non-NaN operand */
        if (!(v <= FLT_MAX)) v = FLT_MAX;
        w[t] = v;
    }
}

/* m_t = A_t / sum(A): Eq. 1 on the fixed-point weights.  The normalisation is a product
 * with the reciprocal of the total, rounded once to fp64 (1 / SA), then the product rounded
 * to fp64 and to fp32: two roundings of 2^-53 against a decision quantum of 2^-36. */
void orc_mass(const float *u, int32_t T, float eps, uint64_t *A, uint64_t *SA, float *m)
{
    float *w = (float *)malloc(sizeof(float) * (size_t)T);
    orc_weights(u, T, eps, w);
    orc_fixed_point(w, T, A, SA);
    const double inv_sa = 1.0 / (double)*SA;
    for (int t = 0; t < T; ++t) m[t] = (float)((double)A[t] * inv_sa);
    free(w);
}

/* ------------------------------------------------------------------------- */
/* Step 2: EMA credit and history-aware mass (Section 3.3, last paragraph)    */
/* ------------------------------------------------------------------------- */

/* c <- lambda c + (1 - lambda) m in fp32; the mass used downstream is
 * beta * m + (1 - beta) * normalize(c), in fp64 on the fixed-point images; the
 * outer normalisation of the paper is implicit because every later threshold is
 * relative to the total.  Output Hm_t = floor(h_t 2^FIX_BITS).  beta == 1 means
 * "credit not used": c is left untouched and h = m. */
void orc_history_mass(const uint64_t *A, uint64_t SA, const float *m, float *credit, int32_t T,
                      float lambda, float beta, uint64_t *Hm)
{
    const double two_f = ldexp(1.0, FIX_BITS);
    const double inv_sa = 1.0 / (double)SA; /* normalisations multiply by the rounded reciprocal */
    if (beta == 1.0f) {
        for (int t = 0; t < T; ++t) Hm[t] = (uint64_t)floor(((double)A[t] * inv_sa) * two_f);
        return;
    }
    const float oml = 1.0f - lambda;
    for (int t = 0; t < T; ++t) {
        const float a = lambda * credit[t];
        const float b = oml * m[t];
        credit[t] = a + b;
    }
    uint64_t *Cq = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)T);
    uint64_t SC = 0;
    orc_fixed_point(credit, T, Cq, &SC);
    const double bd = (double)beta, omb = 1.0 - (double)beta;
    const double inv_sc = (SC > 0) ? 1.0 / (double)SC : 0.0;
    for (int t = 0; t < T; ++t) {
        const double cur = bd * ((double)A[t] * inv_sa);
        const double hist = (SC > 0) ? omb * ((double)Cq[t] * inv_sc) : 0.0;
        Hm[t] = (uint64_t)floor((cur + hist) * two_f);
    }
    free(Cq);
}

/* ------------------------------------------------------------------------- */
/* Step 3: prefix sums, mass-quantile cuts, merge and split                   */
/* ------------------------------------------------------------------------- */

void orc_prefix(const uint64_t *Hm, int32_t T, uint64_t *C)
{
    uint64_t s = 0;
    for (int t = 0; t < T; ++t) { s += Hm[t]; C[t] = s; }
}

/* b_k = min{t : c(t) >= k * Delta}, Delta = 1/S, k = 1..S-1, with 1-based t, and
 * segments [a_i, b_i): in 0-based positions the token that reaches the threshold
 * closes its segment, so the boundary is (position + 1).  Returns the sorted,
 * de-duplicated boundary list including 0 and T; n_bounds-1 raw segments. */
int32_t orc_cuts(const uint64_t *C, int32_t T, int32_t S, int32_t *bounds /* >= S+1 */)
{
    const uint64_t SH = C[T - 1];
    int32_t n = 0;
    bounds[n++] = 0;
    for (int k = 1; k < S; ++k) {
        int p = -1;
        for (int t = 0; t < T; ++t) {
            if (C[t] * (uint64_t)S >= (uint64_t)k * SH) { p = t; break; }
        }
        if (p < 0) continue;
        const int32_t cut = p + 1;
        if (cut > bounds[n - 1] && cut < T) bounds[n++] = cut;
    }
    bounds[n++] = T;
    return n;
}

/* Merge short raw segments forward, fold a short tail into its left neighbour,
 * then split long segments into ceil(len / l_max) pieces whose sizes differ by
 * at most one (larger pieces first).  Returns the number of boundaries written
 * (segments + 1), or -1 if `cap` is too small. */
int32_t orc_merge_split(const int32_t *raw, int32_t n_raw, int32_t l_min, int32_t l_max,
                        int32_t *out, int32_t cap)
{
    const int32_t T = raw[n_raw - 1];
    int32_t *mb = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_raw);
    int32_t nm = 0;
    mb[nm++] = 0;
    for (int i = 1; i < n_raw; ++i) {
        const int32_t e = raw[i];
        if (e == T || e - mb[nm - 1] >= l_min) mb[nm++] = e;
    }
    if (nm > 2 && mb[nm - 1] - mb[nm - 2] < l_min) { mb[nm - 2] = mb[nm - 1]; --nm; }
    int32_t n = 0;
    if (cap < 1) { free(mb); return -1; }
    out[n++] = 0;
    for (int i = 1; i < nm; ++i) {
        const int32_t a = mb[i - 1], len = mb[i] - mb[i - 1];
        int32_t pieces = 1;
        if (l_max > 0 && len > l_max) pieces = (len + l_max - 1) / l_max;
        const int32_t base = len / pieces, extra = len % pieces;
        int32_t pos = a;
        for (int j = 0; j < pieces; ++j) {
            pos += base + (j < extra ? 1 : 0);
            if (n >= cap) { free(mb); return -1; }
            out[n++] = pos;
        }
    }
    free(mb);
    return n;
}

/* ------------------------------------------------------------------------- */
/* Step 4: quotas                                                             */
/* ------------------------------------------------------------------------- */

typedef struct { uint64_t M; int32_t i; } seg_key;

static int by_mass_desc(const void *a, const void *b)
{
    const seg_key *x = (const seg_key *)a, *y = (const seg_key *)b;
    if (x->M != y->M) return x->M > y->M ? -1 : 1;
    return x->i < y->i ? -1 : (x->i > y->i ? 1 : 0);
}

/* Must-keep sizes: sinks first, then as much of the recent suffix as fits. */
void orc_must_keep(int32_t T, int32_t Tk, int32_t n_sink, int32_t n_last, int32_t *ns, int32_t *nl)
{
    int32_t s = n_sink; if (s > Tk) s = Tk; if (s > T) s = T; if (s < 0) s = 0;
    int32_t l = n_last; if (l > Tk - s) l = Tk - s; if (l > T - s) l = T - s; if (l < 0) l = 0;
    *ns = s; *nl = l;
}

/* q_i = q_i^min + round(T_rem * M_i / sum M), clipped to L_i, then the adjustment
 * that makes the quotas sum to the segment budget Bq: a deficit is handed out one
 * token per visit, visiting segments heaviest first (ties: lower index) and
 * cycling while any has room; a surplus is taken back one token per visit,
 * lightest first (ties: higher index), never below q_i^min unless the budget
 * cannot even cover the minima (then a second round goes down to zero). */
void orc_quotas(const uint64_t *C, const int32_t *bounds, int32_t n_seg, int32_t q_min, int32_t Bq,
                int32_t *q)
{
    const uint64_t SH = C[bounds[n_seg] - 1];
    uint64_t *M = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)n_seg);
    int32_t *qmin = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_seg);
    seg_key *ord = (seg_key *)malloc(sizeof(seg_key) * (size_t)n_seg);
    int64_t sum_min = 0;
    for (int i = 0; i < n_seg; ++i) {
        const int32_t a = bounds[i], b = bounds[i + 1], L = b - a;
        M[i] = C[b - 1] - (a > 0 ? C[a - 1] : 0);
        qmin[i] = q_min < L ? q_min : L;
        if (qmin[i] < 0) qmin[i] = 0;
        sum_min += qmin[i];
        ord[i].M = M[i];
        ord[i].i = i;
    }
    const int64_t Trem = (int64_t)Bq - sum_min;
    int64_t sum_q = 0;
    for (int i = 0; i < n_seg; ++i) {
        const int32_t L = bounds[i + 1] - bounds[i];
        int64_t qi = qmin[i];
        if (Trem >= 0) qi += (int64_t)((2 * (uint64_t)Trem * M[i] + SH) / (2 * SH));
        if (qi > L) qi = L;
        q[i] = (int32_t)qi;
        sum_q += qi;
    }
    int64_t Dq = (int64_t)Bq - sum_q;
    qsort(ord, (size_t)n_seg, sizeof(seg_key), by_mass_desc);
    while (Dq > 0) {
        int moved = 0;
        for (int r = 0; r < n_seg && Dq > 0; ++r) { /* (M desc, i asc) */
            const int i = ord[r].i;
            if (q[i] < bounds[i + 1] - bounds[i]) { ++q[i]; --Dq; moved = 1; }
        }
        if (!moved) break;
    }
    for (int pass = 0; pass < 2 && Dq < 0; ++pass) {
        while (Dq < 0) {
            int moved = 0;
            for (int r = n_seg - 1; r >= 0 && Dq < 0; --r) { /* (M asc, i desc) */
                const int i = ord[r].i;
                if (q[i] > (pass == 0 ? qmin[i] : 0)) { --q[i]; ++Dq; moved = 1; }
            }
            if (!moved) break;
        }
    }
    free(M); free(qmin); free(ord);
}

/* ------------------------------------------------------------------------- */
/* Step 5: in-segment top-k, must-keep union, backfill                        */
/* ------------------------------------------------------------------------- */

/* Order-preserving image of an fp32 score; NaN ranks below everything. */
static uint32_t score_key(float x)
{
    uint32_t b;
    memcpy(&b, &x, sizeof b);
    if ((b & 0x7fffffffu) > 0x7f800000u) return 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

typedef struct { uint32_t key; int32_t pos; } tok_key;

static int by_key_desc_pos_asc(const void *a, const void *b)
{
    const tok_key *x = (const tok_key *)a, *y = (const tok_key *)b;
    if (x->key != y->key) return x->key > y->key ? -1 : 1;
    return x->pos < y->pos ? -1 : (x->pos > y->pos ? 1 : 0);
}

/* Keep set of exactly Tk positions, ascending.  Returns the number of backfilled
 * positions, or -1 if the set would exceed Tk (cannot happen when the quotas sum
 * to Tk - ns - nl; the paper's trim branch is therefore unreachable here). */
int32_t orc_select(const float *g, int32_t T, const int32_t *bounds, const int32_t *q, int32_t n_seg,
                   int32_t ns, int32_t nl, int32_t Tk, int32_t *keep_idx)
{
    uint8_t *flag = (uint8_t *)calloc((size_t)T, 1);
    tok_key *buf = (tok_key *)malloc(sizeof(tok_key) * (size_t)T);
    for (int i = 0; i < n_seg; ++i) {
        const int32_t a = bounds[i], b = bounds[i + 1], L = b - a;
        for (int t = 0; t < L; ++t) { buf[t].key = score_key(g[a + t]); buf[t].pos = a + t; }
        qsort(buf, (size_t)L, sizeof(tok_key), by_key_desc_pos_asc);
        for (int j = 0; j < q[i]; ++j) flag[buf[j].pos] = 1;
    }
    for (int t = 0; t < ns; ++t) flag[t] = 1;
    for (int t = T - nl; t < T; ++t) flag[t] = 1;
    int32_t kept = 0;
    for (int t = 0; t < T; ++t) kept += flag[t];
    const int32_t r = Tk - kept;
    if (r < 0) { free(flag); free(buf); return -1; }
    if (r > 0) {
        int32_t n = 0;
        for (int t = 0; t < T; ++t) if (!flag[t]) { buf[n].key = score_key(g[t]); buf[n].pos = t; ++n; }
        qsort(buf, (size_t)n, sizeof(tok_key), by_key_desc_pos_asc);
        for (int j = 0; j < r; ++j) flag[buf[j].pos] = 1;
    }
    int32_t j = 0;
    for (int t = 0; t < T; ++t) if (flag[t]) keep_idx[j++] = t;
    free(flag); free(buf);
    return r;
}

/* ------------------------------------------------------------------------- */
/* Steps 1-5 for one (layer, sequence, KV head)                               */
/* ------------------------------------------------------------------------- */

/* u: usage scores that define the mass; g: base scores used inside segments
 * (may alias u); credit: in/out EMA credit of length >= T (rows travel with
 * their tokens: after selection credit[j] = credit_old[keep_idx[j]] for j < Tk and
 * 0 for Tk <= j < T).  Optional outputs may be NULL.  bounds/quotas need `cap`+1 /
 * `cap` entries.  Returns the number of segments, or a negative error. */
int32_t orc_select_unit(const float *u, const float *g, float *credit, int32_t T, int32_t Tk,
                        const orc_params *prm, int32_t cap, float *mass_out, int32_t *raw_out,
                        int32_t *n_raw_out, int32_t *bounds_out, int32_t *quota_out,
                        int32_t *keep_idx, int32_t *n_backfill_out)
{
    if (T <= Tk || Tk < 1 || prm->n_segments < 1) return -1;
    uint64_t *A = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)T);
    uint64_t *Hm = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)T);
    uint64_t *C = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)T);
    float *m = (float *)malloc(sizeof(float) * (size_t)T);
    int32_t *raw = (int32_t *)malloc(sizeof(int32_t) * (size_t)(prm->n_segments + 1));
    int32_t *bounds = (int32_t *)malloc(sizeof(int32_t) * (size_t)(cap + 1));
    int32_t *q = (int32_t *)malloc(sizeof(int32_t) * (size_t)cap);
    uint64_t SA = 0;
    int32_t ret;

    orc_mass(u, T, prm->eps, A, &SA, m);
    orc_history_mass(A, SA, m, credit, T, prm->ema_lambda, prm->ema_beta, Hm);
    orc_prefix(Hm, T, C);
    int32_t n_raw;
    if (prm->fixed_segments) {
        /* component ablation of the paper: S segments of equal length instead of equal mass,
         * boundary k at floor(k T / S); merge and split then act as usual */
        n_raw = 0;
        raw[n_raw++] = 0;
        for (int k = 1; k < prm->n_segments; ++k) {
            const int32_t cut = (int32_t)(((int64_t)k * T) / prm->n_segments);
            if (cut > raw[n_raw - 1] && cut < T) raw[n_raw++] = cut;
        }
        raw[n_raw++] = T;
    } else {
        n_raw = orc_cuts(C, T, prm->n_segments, raw);
    }
    const int32_t nb = orc_merge_split(raw, n_raw, prm->l_min, prm->l_max, bounds, cap + 1);
    if (nb < 2) { ret = -3; goto done; }
    const int32_t n_seg = nb - 1;
    int32_t ns, nl;
    orc_must_keep(T, Tk, prm->n_sink, prm->n_last, &ns, &nl);
    if (prm->uniform_quotas) {
        /* component ablation of the paper: the budget is shared by segment length, not by mass:
         * the quota routine sees a "mass" of one per token */
        uint64_t *ones = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)T);
        for (int t = 0; t < T; ++t) ones[t] = (uint64_t)t + 1;
        orc_quotas(ones, bounds, n_seg, prm->q_min, Tk - ns - nl, q);
        free(ones);
    } else {
        orc_quotas(C, bounds, n_seg, prm->q_min, Tk - ns - nl, q);
    }
    const int32_t nbf = orc_select(g, T, bounds, q, n_seg, ns, nl, Tk, keep_idx);
    if (nbf < 0) { ret = -4; goto done; }
    if (prm->ema_beta != 1.0f) {
        float *tmp = (float *)malloc(sizeof(float) * (size_t)Tk);
        for (int j = 0; j < Tk; ++j) tmp[j] = credit[keep_idx[j]];
        for (int j = 0; j < Tk; ++j) credit[j] = tmp[j];
        for (int j = Tk; j < T; ++j) credit[j] = 0.0f;
        free(tmp);
    }
    if (mass_out) memcpy(mass_out, m, sizeof(float) * (size_t)T);
    if (raw_out) memcpy(raw_out, raw, sizeof(int32_t) * (size_t)n_raw);
    if (n_raw_out) *n_raw_out = n_raw;
    if (bounds_out) memcpy(bounds_out, bounds, sizeof(int32_t) * (size_t)nb);
    if (quota_out) memcpy(quota_out, q, sizeof(int32_t) * (size_t)n_seg);
    if (n_backfill_out) *n_backfill_out = nbf;
    ret = n_seg;
done:
    free(A); free(Hm); free(C); free(m); free(raw); free(bounds); free(q);
    return ret;
}

/* ------------------------------------------------------------------------- */
/* Step 6: paged head-wise compaction (the two display equations of the       */
/* paged-compaction appendix)                                                 */
/* ------------------------------------------------------------------------- */

/* For compact position j of head h: source slot = pi_old(b, keep_idx[j]) from the
 * sequence's current block-table row, destination slot = pi_new(b, j) from the
 * replacement pages; the head's K row and V row move.  Out of place: source
 * pages are read only. */
void orc_gather_unit(uint16_t *k_pages, uint16_t *v_pages, int64_t num_pages, int32_t page_size,
                     int32_t n_kv_heads, int32_t head_dim, int32_t layer, int32_t h,
                     const int32_t *table_row, const int32_t *dst_row, const int32_t *keep_idx,
                     int32_t Tk)
{
    orc_pool P = {k_pages, num_pages, page_size, n_kv_heads, head_dim};
    for (int j = 0; j < Tk; ++j) {
        const int p = keep_idx[j];
        const int64_t src = row_offset(&P, layer, table_row[p / page_size], p % page_size, h);
        const int64_t dst = row_offset(&P, layer, dst_row[j / page_size], j % page_size, h);
        memcpy(k_pages + dst, k_pages + src, sizeof(uint16_t) * (size_t)head_dim);
        memcpy(v_pages + dst, v_pages + src, sizeof(uint16_t) * (size_t)head_dim);
    }
}
