/*
 * CPU oracle for the MoE routing + load-control path of ID Balancing
 * (arXiv 2609.39137).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, scalar, obviously-correct
 * statement of what the path computes.  It is compiled with
 *   gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
 * and is used by the tests, by the smoke check and by the benchmark's CPU
 * baseline.  It shares no code with the CUDA library and the product never
 * calls it.
 *
 * Two entry families:
 *   "f64"  the definition: fp64 logits from the bf16 operands, libm sigmoid,
 *          full sort.  (Section 2.2, Eq. 2, Eq. 3, Algorithm 1, Eq. 13.)
 *   "f32"  the same chain in the binary32 arithmetic the GPU path computes
 *          in, written operation by operation so that a second
 *          implementation can reproduce every bit.  Starts from fp32 logits.
 *
 * Every function names the passage of the paper it follows.  Where the paper
 * leaves a choice open the choice is stated in the comment ("reading").
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* bf16 <-> binary64.  A bf16 value is the upper 16 bits of a binary32.      */
/* ------------------------------------------------------------------------ */
static double bf16_value(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/*
 * Router logits, Section 2.2: z = W_r x with W_r in R^{E x d}.
 *   x : [T][H] bf16 bit patterns (token-major)
 *   w : [E][H] bf16 bit patterns (one row per expert)
 *   z : [T][E] binary64
 * Each bf16*bf16 product is exact in binary64; the sum runs over h in
 * increasing order.
 */
void oracle_router_logits_f64(const uint16_t *x, const uint16_t *w,
                              int64_t T, int64_t H, int64_t E, double *z)
{
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t e = 0; e < E; ++e) {
            double acc = 0.0;
            for (int64_t h = 0; h < H; ++h)
                acc += bf16_value(x[t * H + h]) * bf16_value(w[e * H + h]);
            z[t * E + e] = acc;
        }
    }
}

/* Expert score, Section 2.2: s_i = sigma(z_i); reading: sigma is the logistic
 * sigmoid (the paper calls the loss-free selection score a "biased sigmoid
 * score", Section 4.3). */
double oracle_sigmoid_f64(double z)
{
    return 1.0 / (1.0 + exp(-z));
}

/* ------------------------------------------------------------------------ */
/* Ordering used by TopK (Eq. 2).  Reading: larger biased score first; equal  */
/* biased scores are ordered by the smaller expert index.                    */
/* ------------------------------------------------------------------------ */
typedef struct { double v; int32_t e; } rank64_t;
typedef struct { float  v; int32_t e; } rank32_t;

static int cmp_rank64(const void *pa, const void *pb)
{
    const rank64_t *a = (const rank64_t *)pa, *b = (const rank64_t *)pb;
    if (a->v > b->v) return -1;
    if (a->v < b->v) return 1;
    return (a->e > b->e) - (a->e < b->e);
}

static int cmp_rank32(const void *pa, const void *pb)
{
    const rank32_t *a = (const rank32_t *)pa, *b = (const rank32_t *)pb;
    if (a->v > b->v) return -1;
    if (a->v < b->v) return 1;
    return (a->e > b->e) - (a->e < b->e);
}

/*
 * Routing in binary64 (Eq. 2 and the sentence after it).
 *   z     : [T][E] logits
 *   b     : [E] bias (binary32 state, widened exactly)
 *   idx   : [T][K] selected experts, ordered by descending biased score
 *   gate  : [T][K] combination weights = s_k / sum of the selected s (no bias)
 *   alpha : [T] (K+1)-th largest biased score (Section 2.3, Quantile
 *           Balancing cutoff); NaN when K == E.  May be NULL.
 *   gap   : [T] K-th minus (K+1)-th largest biased score; +inf when K == E.
 *           May be NULL.
 * Returns 0, or -1 on a bad argument / allocation failure.
 */
int oracle_route_f64(const double *z, const float *b, int64_t T, int64_t E,
                     int64_t K, int32_t *idx, double *gate, double *alpha,
                     double *gap)
{
    if (K < 1 || K > E) return -1;
    rank64_t *r = (rank64_t *)malloc((size_t)E * sizeof *r);
    double *s = (double *)malloc((size_t)E * sizeof *s);
    if (!r || !s) { free(r); free(s); return -1; }
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t e = 0; e < E; ++e) {
            s[e] = oracle_sigmoid_f64(z[t * E + e]);
            r[e].v = s[e] + (double)b[e];
            r[e].e = (int32_t)e;
        }
        qsort(r, (size_t)E, sizeof *r, cmp_rank64);
        double denom = 0.0;
        for (int64_t k = 0; k < K; ++k) denom += s[r[k].e];
        for (int64_t k = 0; k < K; ++k) {
            idx[t * K + k] = r[k].e;
            gate[t * K + k] = s[r[k].e] / denom;
        }
        if (alpha) alpha[t] = (K < E) ? r[K].v : NAN;
        if (gap) gap[t] = (K < E) ? r[K - 1].v - r[K].v : INFINITY;
    }
    free(r); free(s);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* binary32 chain.  IEEE-754 binary32, round-to-nearest-even, no contraction  */
/* except where fmaf is written, no flush-to-zero.                           */
/* ------------------------------------------------------------------------ */

/*
 * Logistic sigmoid in binary32 (score of Section 2.2), fixed operation order:
 *   t = z * (-log2 e)                       one multiply
 *   t = clamp(t, -125, 125)                 keeps 2^n * p a normal number
 *   n = nearest integer to t, ties to even
 *   f = t - n                               exact, |f| <= 1/2
 *   p = 2^f by the degree-6 Taylor polynomial in f*ln2, Horner with fmaf
 *   u = p * 2^n                             exponent-field addition
 *   s = 1 / (1 + u)                         one add, one IEEE divide
 * The absolute error against the real sigmoid is below 2e-7.
 */
float oracle_sigmoid_f32(float z)
{
    const float c6 = 1.5403530e-4f, c5 = 1.3333558e-3f, c4 = 9.6181291e-3f,
                c3 = 5.5504109e-2f, c2 = 2.4022651e-1f, c1 = 6.9314718e-1f,
                c0 = 1.0f;
    float t = z * -1.44269504f;
    t = fminf(fmaxf(t, -125.0f), 125.0f);
    float n = rintf(t);
    float f = t - n;
    float p = c6;
    p = fmaf(p, f, c5);
    p = fmaf(p, f, c4);
    p = fmaf(p, f, c3);
    p = fmaf(p, f, c2);
    p = fmaf(p, f, c1);
    p = fmaf(p, f, c0);
    uint32_t bits;
    memcpy(&bits, &p, sizeof bits);
    bits += (uint32_t)(int32_t)n << 23;   /* wraps mod 2^32 for n < 0 */
    float u;
    memcpy(&u, &bits, sizeof u);
    float d = 1.0f + u;
    return 1.0f / d;
}

void oracle_sigmoid_f32_array(const float *z, int64_t n, float *s)
{
    for (int64_t i = 0; i < n; ++i) s[i] = oracle_sigmoid_f32(z[i]);
}

/*
 * Routing in binary32 (Eq. 2) from fp32 logits.
 *   v_e = sigmoid_f32(z_e) + b_e            one add
 *   order: v descending, ties by ascending e (floats compared as values)
 *   gate: D = ((s_0 + s_1) + s_2) + ... in output order, w_k = s_k / D;
 *         D == 0 gives 1/K each.
 *   alpha[t] = v of rank K+1 (may be NULL; NaN if K == E)
 */
int oracle_route_f32(const float *z, const float *b, int64_t T, int64_t E,
                     int64_t K, int32_t *idx, float *gate, float *alpha)
{
    if (K < 1 || K > E) return -1;
    rank32_t *r = (rank32_t *)malloc((size_t)E * sizeof *r);
    float *s = (float *)malloc((size_t)E * sizeof *s);
    if (!r || !s) { free(r); free(s); return -1; }
    for (int64_t t = 0; t < T; ++t) {
        for (int64_t e = 0; e < E; ++e) {
            s[e] = oracle_sigmoid_f32(z[t * E + e]);
            r[e].v = s[e] + b[e];
            r[e].e = (int32_t)e;
        }
        qsort(r, (size_t)E, sizeof *r, cmp_rank32);
        float denom = s[r[0].e];
        for (int64_t k = 1; k < K; ++k) denom = denom + s[r[k].e];
        for (int64_t k = 0; k < K; ++k) {
            idx[t * K + k] = r[k].e;
            gate[t * K + k] = (denom == 0.0f) ? 1.0f / (float)K
                                              : s[r[k].e] / denom;
        }
        if (alpha) alpha[t] = (K < E) ? r[K].v : NAN;
    }
    free(r); free(s);
    return 0;
}

/*
 * Load counts, Section 2.2 / Algorithm 1 line 4: n_i = number of tokens
 * assigned to expert i.  ADDS to n (microbatches accumulate).
 * Returns -1 if an index is outside [0, E).
 */
int oracle_load_counts(const int32_t *idx, int64_t T, int64_t K, int64_t E,
                       int64_t *n)
{
    for (int64_t i = 0; i < T * K; ++i) {
        if (idx[i] < 0 || idx[i] >= E) return -1;
        n[idx[i]] += 1;
    }
    return 0;
}

/*
 * Uniform target and normalised error, Eq. 3 / Algorithm 1 lines 5-7:
 *   nbar = (1/E) sum n_i ;  e_i = (nbar - n_i) / nbar
 * computed in binary64 and rounded once to binary32.
 * Returns -1 when sum n == 0 (the paper requires a non-empty batch).
 */
int oracle_load_error(const int64_t *n, int64_t E, float *e)
{
    int64_t total = 0;
    for (int64_t i = 0; i < E; ++i) total += n[i];
    if (total <= 0) return -1;
    double nbar = (double)total / (double)E;
    for (int64_t i = 0; i < E; ++i)
        e[i] = (float)((nbar - (double)n[i]) / nbar);
    return 0;
}

/*
 * Zero-mean centring, Algorithm 1 line 13 / Eq. 12 second line:
 *   b_i <- b_i - (1/E) sum_j b_j.
 * Reading (summation order is not fixed by the paper): the sum is taken in
 * binary64 over the values padded with zeros to 1024 entries, pairwise with
 * strides 512, 256, ..., 1 (y[i] += y[i + stride]); mean = (float)(y[0] / E);
 * then one binary32 subtraction per expert.  Requires E <= 1024.
 */
int oracle_center(float *b, int64_t E)
{
    double y[1024];
    if (E < 1 || E > 1024) return -1;
    for (int64_t i = 0; i < 1024; ++i) y[i] = (i < E) ? (double)b[i] : 0.0;
    for (int64_t stride = 512; stride >= 1; stride /= 2)
        for (int64_t i = 0; i < stride; ++i) y[i] = y[i] + y[i + stride];
    float mean = (float)(y[0] / (double)E);
    for (int64_t i = 0; i < E; ++i) b[i] = b[i] - mean;
    return 0;
}

/*
 * ID Balancing update for one layer, Algorithm 1 lines 8-13 (Eq. 9-12), in
 * binary32:
 *   de   = e - e_prev
 *   g    = 1 iff e_prev * de > 0 as real numbers, i.e. e_prev and de are both
 *          positive or both negative (no product is formed, so tiny values
 *          cannot underflow the test)
 *   b    = (b + Ki * e) + (g ? Kd * de : 0)
 *   e_prev <- e
 *   centre if `center` is non-zero.
 * gate_out (may be NULL) receives g per expert.
 */
int oracle_id_update(float *b, float *e_prev, const float *e, int64_t E,
                     float ki, float kd, int center, int32_t *gate_out)
{
    for (int64_t i = 0; i < E; ++i) {
        float de = e[i] - e_prev[i];
        int g = (e_prev[i] > 0.0f && de > 0.0f) ||
                (e_prev[i] < 0.0f && de < 0.0f);
        float t1 = ki * e[i];
        float t2 = g ? kd * de : 0.0f;
        b[i] = (b[i] + t1) + t2;
        e_prev[i] = e[i];
        if (gate_out) gate_out[i] = g;
    }
    return center ? oracle_center(b, E) : 0;
}

/*
 * DeepSeek loss-free update = fixed-step integral control, Eq. 5:
 *   b <- b + eta * sign(e), sign(0) = 0.  Not centred unless asked
 *   (Section 3 notes that this update lets the common component drift).
 * e_prev is kept up to date so that a controller switch stays well defined.
 */
int oracle_fixed_step_update(float *b, float *e_prev, const float *e,
                             int64_t E, float eta, int center)
{
    for (int64_t i = 0; i < E; ++i) {
        float step = (e[i] > 0.0f) ? eta : (e[i] < 0.0f) ? -eta : 0.0f;
        b[i] = b[i] + step;
        e_prev[i] = e[i];
    }
    return center ? oracle_center(b, E) : 0;
}

static int cmp_float(const void *pa, const void *pb)
{
    float a = *(const float *)pa, b = *(const float *)pb;
    return (a > b) - (a < b);
}

/*
 * Quantile Balancing target, Eq. 6-7:
 *   Q_j = - quantile_{1-K/E}( { S_ij - alpha_i }_i ),
 * S_ij = sigmoid_f32(z_ij) the unbiased score, alpha_i the (K+1)-th largest
 * biased score of token i.  Reading (the quantile estimator is not fixed by
 * the paper): nearest rank without interpolation, r = m - floor(m*K/E)
 * clamped to [1, m]; the quantile is the r-th smallest margin, so that with
 * distinct margins exactly floor(m*K/E) tokens lie strictly above it.
 *   z     : [m][E] fp32 logits, alpha : [m], Q : [E]
 */
int oracle_quantile_target(const float *z, const float *alpha, int64_t m,
                           int64_t E, int64_t K, float *Q)
{
    if (m < 1) return -1;
    float *d = (float *)malloc((size_t)m * sizeof *d);
    if (!d) return -1;
    int64_t r = m - (m * K) / E;
    if (r < 1) r = 1;
    if (r > m) r = m;
    for (int64_t j = 0; j < E; ++j) {
        for (int64_t i = 0; i < m; ++i)
            d[i] = oracle_sigmoid_f32(z[i * E + j]) - alpha[i];
        qsort(d, (size_t)m, sizeof *d, cmp_float);
        Q[j] = -d[r - 1];
    }
    free(d);
    return 0;
}

/*
 * Quantile Balancing target estimated from a per-expert margin histogram
 * (footnote to Eq. 7, Section 2.3: "at scale" the quantile is estimated from
 * such a histogram).  The paper fixes neither bins nor range nor the rule
 * inside a bin -- PARITY UNPINNED against the paper; the reading taken here:
 *   B uniform bins over [-range, +range), bin width h = 2*range/B;
 *   margin d = sigmoid_f32(z_ij) - alpha_i in binary32 (as in the exact form);
 *   bin k = floor((d + range) * inv_h) with inv_h = (float)B / (2*range), both
 *   operations rounded to binary32, clamped to [0, B-1] (margins outside the
 *   range count in the end bins);
 *   same nearest rank as the exact form, r = m - floor(m*K/E) in [1, m];
 *   k* = the bin that holds the r-th smallest margin (below = count of the
 *   bins before it, cnt = its own count); estimate by linear interpolation
 *   at the middle of the r-th margin's share of the bin, in binary64,
 *     est = -range + (k* + ((r - below) - 0.5) / cnt) * h,   Q_j = -(float)est.
 * Since the exact r-th smallest margin lies in bin k* too, |est - exact| < h
 * whenever that margin is inside the range.  hist (may be NULL) receives the
 * counts, [E][B].
 */
int oracle_quantile_target_hist(const float *z, const float *alpha, int64_t m,
                                int64_t E, int64_t K, int64_t B, float range,
                                float *Q, int64_t *hist)
{
    if (m < 1 || B < 1 || !(range > 0.0f)) return -1;
    int64_t *cnt = (int64_t *)malloc((size_t)B * sizeof *cnt);
    if (!cnt) return -1;
    int64_t r = m - (m * K) / E;
    if (r < 1) r = 1;
    if (r > m) r = m;
    const float inv_h = (float)B / (2.0f * range);
    const double h = 2.0 * (double)range / (double)B;
    for (int64_t j = 0; j < E; ++j) {
        for (int64_t k = 0; k < B; ++k) cnt[k] = 0;
        for (int64_t i = 0; i < m; ++i) {
            float d = oracle_sigmoid_f32(z[i * E + j]) - alpha[i];
            float shifted = d + range;
            float u = shifted * inv_h;
            int64_t k = 0;
            if (u >= 0.0f) {
                float fl = floorf(u);
                k = (fl >= (float)B) ? B - 1 : (int64_t)fl;
            }
            cnt[k] += 1;
        }
        int64_t below = 0, kstar = 0;
        for (int64_t k = 0; k < B; ++k) {
            if (r <= below + cnt[k]) { kstar = k; break; }
            below += cnt[k];
        }
        double inside = ((double)(r - below) - 0.5) / (double)cnt[kstar];
        double est = -(double)range + ((double)kstar + inside) * h;
        Q[j] = -(float)est;
        if (hist)
            for (int64_t k = 0; k < B; ++k) hist[j * B + k] = cnt[k];
    }
    free(cnt);
    return 0;
}

/*
 * Quantile Balancing update with the diagnostic EMA of Section 3:
 *   b <- rho * b + (1 - rho) * Q, 0 <= rho < 1; rho = 0 stores Q unchanged.
 * binary32: (rho * b) + ((1 - rho) * Q), no fused multiply-add.
 */
int oracle_quantile_update(float *b, float *e_prev, const float *e,
                           const float *Q, int64_t E, float rho, int center)
{
    for (int64_t j = 0; j < E; ++j) {
        if (rho == 0.0f) {
            b[j] = Q[j];
        } else {
            float keep = rho * b[j];
            float take = (1.0f - rho) * Q[j];
            b[j] = keep + take;
        }
        e_prev[j] = e[j];
    }
    return center ? oracle_center(b, E) : 0;
}

/*
 * Load-violation metrics, Eq. 13:
 *   MaxVio = (max n - nbar) / nbar ;  MinVio = (nbar - min n) / nbar
 * in binary64, rounded once to binary32.
 */
int oracle_violations(const int64_t *n, int64_t E, float *maxvio,
                      float *minvio)
{
    int64_t total = 0, hi = n[0], lo = n[0];
    for (int64_t i = 0; i < E; ++i) {
        total += n[i];
        if (n[i] > hi) hi = n[i];
        if (n[i] < lo) lo = n[i];
    }
    if (total <= 0) return -1;
    double nbar = (double)total / (double)E;
    *maxvio = (float)(((double)hi - nbar) / nbar);
    *minvio = (float)((nbar - (double)lo) / nbar);
    return 0;
}

/*
 * Load-control diagnostics the paper plots (Section 3 figure captions, Section 4.3), per layer:
 *   gate_frac     fraction of experts whose worsening gate g_i is open (Eq. 11)
 *   busiest_share share of all token assignments that went to the busiest 10 % of
 *                 the experts (balanced value 0.10).  Reading: "10 % of the experts"
 *                 is m = E/10 rounded to the nearest integer (at least 1).
 *   inactive      fraction of experts that received no token
 *   bias_drift    mean absolute bias change (1/E) sum |b_new - b_old|
 * All in binary64, rounded once to binary32.  out[4] in the order above.
 */
static int cmp_i64_desc(const void *pa, const void *pb)
{
    int64_t a = *(const int64_t *)pa, b = *(const int64_t *)pb;
    return (a < b) - (a > b);
}

int oracle_load_diagnostics(const int64_t *n, const int32_t *gate, const float *b_old,
                            const float *b_new, int64_t E, float *out)
{
    int64_t *sorted = (int64_t *)malloc((size_t)E * sizeof *sorted);
    if (!sorted) return -1;
    int64_t total = 0, open_gates = 0, empty = 0;
    double drift = 0.0;
    for (int64_t i = 0; i < E; ++i) {
        sorted[i] = n[i];
        total += n[i];
        open_gates += gate[i] ? 1 : 0;
        empty += (n[i] == 0);
        drift += fabs((double)b_new[i] - (double)b_old[i]);
    }
    if (total <= 0) { free(sorted); return -1; }
    qsort(sorted, (size_t)E, sizeof *sorted, cmp_i64_desc);
    int64_t m = (E + 5) / 10;
    if (m < 1) m = 1;
    int64_t top = 0;
    for (int64_t i = 0; i < m; ++i) top += sorted[i];
    out[0] = (float)((double)open_gates / (double)E);
    out[1] = (float)((double)top / (double)total);
    out[2] = (float)((double)empty / (double)E);
    out[3] = (float)(drift / (double)E);
    free(sorted);
    return 0;
}

/*
 * Top-K gating-score entropy (Section 4.3): H = - sum_{k<K} w_k ln w_k in nats,
 * w the normalised combination weights of a token; returns the mean over the
 * T tokens (0 ln 0 = 0).  gate : [T][K] binary32.
 */
double oracle_gate_entropy_mean(const float *gate, int64_t T, int64_t K)
{
    double sum = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        double h = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double w = (double)gate[t * K + k];
            if (w > 0.0) h -= w * log(w);
        }
        sum += h;
    }
    return sum / (double)T;
}

/*
 * Full-pool selection-score entropy of one token (Section 4.3):
 * H = - sum_e p_e ln p_e in nats (0 ln 0 = 0), where
 *   kind 0 (bias-controlled methods): p_e = c_e / sum_j c_j with
 *           c_e = max(sigmoid(z_e) + b_e, 0), the biased score clamped at zero;
 *   kind 1 (auxiliary loss): p_e = softmax_e(z) = exp(z_e) / sum_j exp(z_j),
 *           written as the definition (binary64 exp cannot overflow for
 *           |z| < 700; router logits are far inside).
 * A token whose clamped scores are all zero has no distribution; H = 0 then.
 * z : [E] binary32 logits, b : [E] binary32 bias (ignored for kind 1).
 */
double oracle_full_pool_entropy(const float *z, const float *b, int64_t E, int kind)
{
    double total = 0.0;
    for (int64_t e = 0; e < E; ++e) {
        double c;
        if (kind == 0) {
            c = oracle_sigmoid_f64((double)z[e]) + (double)b[e];
            if (c < 0.0) c = 0.0;
        } else {
            c = exp((double)z[e]);
        }
        total += c;
    }
    if (!(total > 0.0)) return 0.0;
    double h = 0.0;
    for (int64_t e = 0; e < E; ++e) {
        double c;
        if (kind == 0) {
            c = oracle_sigmoid_f64((double)z[e]) + (double)b[e];
            if (c < 0.0) c = 0.0;
        } else {
            c = exp((double)z[e]);
        }
        double p = c / total;
        if (p > 0.0) h -= p * log(p);
    }
    return h;
}

/* Mean of oracle_full_pool_entropy over the T tokens of z [T][E]. */
double oracle_full_pool_entropy_mean(const float *z, const float *b, int64_t T, int64_t E, int kind)
{
    double sum = 0.0;
    for (int64_t t = 0; t < T; ++t) sum += oracle_full_pool_entropy(z + t * E, b, E, kind);
    return sum / (double)T;
}

/*
 * Statistics of the auxiliary balancing loss (Eq. 8), forward only:
 *   f_i = n_i / T          fraction of the T tokens assigned to expert i,
 *   P_i = (1/T) sum_x softmax_i(W_r x)   mean router probability,
 *   aux = sum_i f_i P_i    (the coefficient alpha of Eq. 8 is left to the caller).
 * z : [T][E] binary32 logits, n : [E] counts of the same T tokens.
 */
void oracle_aux_loss_stats(const float *z, int64_t T, int64_t E, const int64_t *n,
                           double *f, double *P, double *aux)
{
    for (int64_t e = 0; e < E; ++e) P[e] = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        const float *zt = z + t * E;
        double total = 0.0;
        for (int64_t e = 0; e < E; ++e) total += exp((double)zt[e]);
        for (int64_t e = 0; e < E; ++e) P[e] += exp((double)zt[e]) / total;
    }
    double a = 0.0;
    for (int64_t e = 0; e < E; ++e) {
        P[e] /= (double)T;
        f[e] = (double)n[e] / (double)T;
        a += f[e] * P[e];
    }
    *aux = a;
}

/*
 * One whole routing pass of the definition for a slice of tokens: logits,
 * scores, biased top-K, gates and load counts (Section 2.2, Algorithm 1
 * lines 3-4).  Convenience for timing and for tests; it only chains the
 * functions above.  z_scratch : [T][E] binary64 work array.
 */
int oracle_route_tokens_f64(const uint16_t *x, const uint16_t *w,
                            const float *b, int64_t T, int64_t H, int64_t E,
                            int64_t K, double *z_scratch, int32_t *idx,
                            double *gate, double *alpha, double *gap,
                            int64_t *n)
{
    oracle_router_logits_f64(x, w, T, H, E, z_scratch);
    if (oracle_route_f64(z_scratch, b, T, E, K, idx, gate, alpha, gap))
        return -1;
    return oracle_load_counts(idx, T, K, E, n);
}
