/*
 * gg_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, fp64 CPU statement of the per-tensor generalized-Gaussian (GG)
 * pass: moments, moment-ratio fit, distribution penalty with its elementwise
 * gradient, floor quantiser with symbol histogram and empirical entropy, and
 * counter-based GG sampling.  It exists so that the CUDA library can be checked
 * against something written straight from the definitions.  It shares no code,
 * header, table or constant generator with the CUDA path, and only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Letters (the paper's Eq. 1 writes the shape as nu and the scale as beta; this
 * code uses the letters of the library's interface):
 *     beta  = shape,   alpha = scale,   location = 0,
 *     f(x) = beta / (2 alpha Gamma(1/beta)) * exp(-(|x|/alpha)^beta)      [Eq. 1]
 *
 * Every input array is fp32 (a bf16 tensor is widened exactly by the caller);
 * all arithmetic below is fp64 (sums: x87 long double), except where the
 * quantiser is DEFINED in fp32.
 *
 * Pin status (tests/test_oracle_*.py): every function here is pinned to closed
 * forms, multi-precision evaluation, brute force or statistical identities.
 * Nothing from the paper's Tables 1-4 / Figures 1-4 can be reproduced without
 * its models and datasets: for those, parity unpinned.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC gg_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#include <stdlib.h>

#define GGO_BETA_LO 0.05
#define GGO_BETA_HI 20.0

#define GGO_FLAG_DEGENERATE      1u   /* n == 0 or sum of squares == 0      */
#define GGO_FLAG_BETA_CLAMPED_LO 2u   /* moment ratio below rho(GGO_BETA_LO) */
#define GGO_FLAG_BETA_CLAMPED_HI 4u   /* moment ratio above rho(GGO_BETA_HI) */
#define GGO_FLAG_NONFINITE       8u   /* an input was inf or nan             */

/* ---------------------------------------------------------------- Eq. 1-5 */

/* ln of the moment ratio rho(beta) = (E|x|)^2 / E[x^2] of a zero-mean GG:
 * E|x| = alpha Gamma(2/beta)/Gamma(1/beta), E[x^2] = alpha^2 Gamma(3/beta)/Gamma(1/beta)
 * (the second is the paper's variance formula, Eq. 3), so
 * rho = Gamma(2/beta)^2 / (Gamma(1/beta) Gamma(3/beta)). */
double ggo_log_rho(double beta)
{
    return 2.0 * lgamma(2.0 / beta) - lgamma(1.0 / beta) - lgamma(3.0 / beta);
}

double ggo_rho(double beta) { return exp(ggo_log_rho(beta)); }

/* Eq. 2: scale from standard deviation, alpha = sigma sqrt(Gamma(1/beta)/Gamma(3/beta)). */
double ggo_alpha_from_std(double sigma, double beta)
{
    return sigma * exp(0.5 * (lgamma(1.0 / beta) - lgamma(3.0 / beta)));
}

/* Eq. 3: variance alpha^2 Gamma(3/beta)/Gamma(1/beta). */
double ggo_variance(double alpha, double beta)
{
    return alpha * alpha * exp(lgamma(3.0 / beta) - lgamma(1.0 / beta));
}

/* First absolute moment alpha Gamma(2/beta)/Gamma(1/beta) (integrate Eq. 1 against |x|). */
double ggo_mean_abs(double alpha, double beta)
{
    return alpha * exp(lgamma(2.0 / beta) - lgamma(1.0 / beta));
}

/* Differential entropy of Eq. 1 in nats: -E[ln f] = 1/beta + ln(2 alpha Gamma(1/beta)/beta),
 * using E[(|x|/alpha)^beta] = 1/beta. */
double ggo_diff_entropy_nats(double alpha, double beta)
{
    return 1.0 / beta + log(2.0 * alpha / beta) + lgamma(1.0 / beta);
}

/* Eq. 4-5, the GG initialisation rule: scale of W^{d_in x d_out} is
 * sqrt(xi/d_in * Gamma(1/beta)/Gamma(3/beta)); xi = 1 (none/sigmoid), 2 (ReLU),
 * 2/(1+k^2) (leaky ReLU of slope k). */
double ggo_init_alpha(int64_t d_in, double xi, double beta)
{
    return sqrt(xi / (double)d_in * exp(lgamma(1.0 / beta) - lgamma(3.0 / beta)));
}

/* --------------------------------------------------------------- moments */

/* S1 = sum |x_i|, S2 = sum x_i^2 over the FINITE entries, count n = all entries. */
void ggo_moments(const float *x, int64_t n, double *sum_abs, double *sum_sq,
                 int64_t *n_nonfinite)
{
    long double s1 = 0.0L, s2 = 0.0L;
    int64_t bad = 0;
    for (int64_t i = 0; i < n; ++i) {
        double v = (double)x[i];
        if (!isfinite(v)) { ++bad; continue; }
        s1 += (long double)fabs(v);
        s2 += (long double)v * (long double)v;
    }
    *sum_abs = (double)s1;
    *sum_sq = (double)s2;
    *n_nonfinite = bad;
}

/* ------------------------------------------------------------------- fit */

/* Moment-ratio fit.  r = (S1/n)^2 / (S2/n); rho is strictly increasing in
 * beta from 0 to 3/4, so rho(beta) = r has one root: bisection on
 * [GGO_BETA_LO, GGO_BETA_HI] to a relative width of 1e-14.  The scale then
 * follows Eq. 2 with sigma^2 = S2/n.  Returns the flag word. */
uint32_t ggo_fit_from_moments(double sum_abs, double sum_sq, int64_t n,
                              int64_t n_nonfinite, double *beta, double *alpha)
{
    uint32_t flags = n_nonfinite > 0 ? GGO_FLAG_NONFINITE : 0u;
    if (n <= 0 || !(sum_sq > 0.0)) {
        *beta = 0.0;
        *alpha = 0.0;
        return flags | GGO_FLAG_DEGENERATE;
    }
    double m1 = sum_abs / (double)n;
    double m2 = sum_sq / (double)n;
    double log_r = log(m1 * m1 / m2);
    double b;
    if (log_r <= ggo_log_rho(GGO_BETA_LO)) {
        b = GGO_BETA_LO;
        flags |= GGO_FLAG_BETA_CLAMPED_LO;
    } else if (log_r >= ggo_log_rho(GGO_BETA_HI)) {
        b = GGO_BETA_HI;
        flags |= GGO_FLAG_BETA_CLAMPED_HI;
    } else {
        double lo = GGO_BETA_LO, hi = GGO_BETA_HI;
        while (hi - lo > 1e-14 * lo) {
            double mid = 0.5 * (lo + hi);
            if (mid <= lo || mid >= hi) break;
            if (ggo_log_rho(mid) < log_r) lo = mid; else hi = mid;
        }
        b = 0.5 * (lo + hi);
    }
    *beta = b;
    *alpha = ggo_alpha_from_std(sqrt(m2), b);
    return flags;
}

/* --------------------------------------------------- penalty and gradient */

/* GG distribution penalty P = lambda * sum (|x_i|/alpha)^beta  (lambda times the
 * negative log-likelihood of Eq. 1 without its constants) and its gradient
 * g_i = lambda beta sign(x_i) |x_i|^(beta-1) / alpha^beta, with g = 0 at x = 0.
 * grad may be NULL.  beta <= 0 or alpha <= 0 (a degenerate fit) gives zeros. */
void ggo_penalty_grad(const float *x, int64_t n, double beta, double alpha,
                      double lambda, double *grad, double *penalty)
{
    if (!(beta > 0.0) || !(alpha > 0.0)) {
        if (grad) for (int64_t i = 0; i < n; ++i) grad[i] = 0.0;
        *penalty = 0.0;
        return;
    }
    long double p = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        double ax = fabs((double)x[i]);
        if (ax != 0.0) p += (long double)pow(ax / alpha, beta);
    }
    *penalty = lambda * (double)p;
    if (!grad) return;
    double alpha_pow_beta = pow(alpha, beta);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double v = (double)x[i];
        double ax = fabs(v);
        double g = 0.0;
        if (ax != 0.0) {
            g = lambda * beta * pow(ax, beta - 1.0) / alpha_pow_beta;
            if (v < 0.0) g = -g;
        }
        grad[i] = g;
    }
}

/* ------------------------------------------- quantiser, histogram, entropy */

/* The quantiser's forward value is a floor (the straight-through form
 * x - sg(x - floor(x)) evaluates to floor(x)); the step need not be a power of
 * two, so the scaling is DEFINED in fp32 to make the symbol unique:
 *     inv = (float)(1.0 / (double)step);   t = fl32( x * inv );
 *     q   = clamp( floor(t), qmin, qmax ).
 * hist has qmax-qmin+1 bins and is ADDED to; clamped[0]/[1] count the symbols
 * moved up to qmin / down to qmax.  NaN inputs are skipped. */
void ggo_quantise_hist(const float *x, int64_t n, float step, int32_t qmin,
                       int32_t qmax, uint64_t *hist, uint64_t *clamped)
{
    const float inv = (float)(1.0 / (double)step);
    for (int64_t i = 0; i < n; ++i) {
        const float t = x[i] * inv;   /* one fp32 multiply, rounded to fp32 */
        double f = floor((double)t);
        if (isnan(f)) continue;
        int32_t q;
        if (f < (double)qmin) { q = qmin; clamped[0] += 1; }
        else if (f > (double)qmax) { q = qmax; clamped[1] += 1; }
        else q = (int32_t)f;
        hist[q - qmin] += 1;
    }
}

/* The same symbols, one per element (for element-wise checks). */
void ggo_quantise(const float *x, int64_t n, float step, int32_t qmin,
                  int32_t qmax, int32_t *q_out)
{
    const float inv = (float)(1.0 / (double)step);
    for (int64_t i = 0; i < n; ++i) {
        const float t = x[i] * inv;   /* one fp32 multiply, rounded to fp32 */
        double f = floor((double)t);
        int32_t q;
        if (isnan(f)) q = 0;
        else if (f < (double)qmin) q = qmin;
        else if (f > (double)qmax) q = qmax;
        else q = (int32_t)f;
        q_out[i] = q;
    }
}

/* Empirical entropy of a count table in bits per symbol:
 * H = log2 N - (1/N) sum_{c>0} c log2 c,  N = sum c;  N = 0 gives 0. */
double ggo_entropy_bits(const uint64_t *hist, int64_t n_bins)
{
    long double total = 0.0L, acc = 0.0L;
    for (int64_t k = 0; k < n_bins; ++k) {
        if (hist[k] == 0) continue;
        double c = (double)hist[k];
        total += (long double)c;
        acc += (long double)(c * log2(c));
    }
    if (total == 0.0L) return 0.0;
    return log2((double)total) - (double)(acc / total);
}

/* -------------------------------------------------------------- sampling */

/* Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11): a keyed
 * bijection of a 128-bit counter.  One round multiplies counter words 0 and 2
 * by two fixed odd constants, keeps both halves of each 64-bit product, and
 * mixes the high halves with the other counter words and the key; the key
 * advances by the golden-ratio / sqrt(3)-1 Weyl constants between rounds. */
void ggo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* 32 random bits -> a uniform in the open interval (0,1): (r + 1/2) 2^-32. */
static double ggo_u01(uint32_t r) { return ((double)r + 0.5) * (1.0 / 4294967296.0); }

#define GGO_SAMPLE_MAX_ATTEMPTS 64u
#define GGO_TWO_PI 6.283185307179586476925286766559

/* One GG(0, alpha, beta) variate for element `index` of tensor `tensor_id`.
 *
 * If G ~ Gamma(1/beta, 1) and s = +-1 with equal probability then
 * s alpha G^(1/beta) has the density of Eq. 1 (change of variable y = (|x|/alpha)^beta).
 * G is drawn by the Marsaglia-Tsang method (2000): with a' = a (a >= 1) or a+1
 * (a < 1), d = a' - 1/3, c = 1/sqrt(9 d): draw z ~ N(0,1), v = (1 + c z)^3;
 * reject if v <= 0; accept if ln u < z^2/2 + d (1 - v + ln v); then G = d v, and
 * for a < 1 multiply by u'^(1/a) with a fresh uniform u'.
 * Randomness is counter-based: attempt t uses the Philox block with counter
 * (index_lo, index_hi, t, tensor_id) and key (seed_lo, seed_hi): words 0,1 make
 * z by Box-Muller, word 2 is the acceptance uniform.  The block with
 * t = 0xFFFFFFFF gives the sign (top bit of word 0) and the a < 1 uniform
 * (word 1).  attempts_out (may be NULL) receives the attempts used; if all
 * GGO_SAMPLE_MAX_ATTEMPTS fail the value is 0 and attempts is MAX+1. */
double ggo_sample_one(double beta, double alpha, uint64_t seed, uint32_t tensor_id,
                      uint64_t index, uint32_t *attempts_out)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t ctr[4] = { (uint32_t)index, (uint32_t)(index >> 32), 0u, tensor_id };
    uint32_t r[4];
    double a = 1.0 / beta;
    double a1 = a >= 1.0 ? a : a + 1.0;
    double d = a1 - 1.0 / 3.0;
    double c = 1.0 / sqrt(9.0 * d);
    double G = 0.0;
    uint32_t t;
    int accepted = 0;
    for (t = 0; t < GGO_SAMPLE_MAX_ATTEMPTS; ++t) {
        ctr[2] = t;
        ggo_philox4x32_10(ctr, key, r);
        double z = sqrt(-2.0 * log(ggo_u01(r[0]))) * cos(GGO_TWO_PI * ggo_u01(r[1]));
        double w = 1.0 + c * z;
        if (w <= 0.0) continue;
        double v = w * w * w;
        if (log(ggo_u01(r[2])) < 0.5 * z * z + d * (1.0 - v + log(v))) {
            G = d * v;
            accepted = 1;
            break;
        }
    }
    if (attempts_out) *attempts_out = accepted ? t + 1u : GGO_SAMPLE_MAX_ATTEMPTS + 1u;
    if (!accepted) return 0.0;
    ctr[2] = 0xFFFFFFFFu;
    ggo_philox4x32_10(ctr, key, r);
    if (a < 1.0) G *= pow(ggo_u01(r[1]), 1.0 / a);
    double x = alpha * pow(G, 1.0 / beta);
    return (r[0] & 0x80000000u) ? -x : x;
}

/* n variates, elements index0 .. index0+n-1, as fp64 (the caller rounds to the
 * storage type).  attempts (uint8 per element) may be NULL. */
void ggo_sample(double beta, double alpha, uint64_t seed, uint32_t tensor_id,
                uint64_t index0, int64_t n, double *out, uint8_t *attempts)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        uint32_t att;
        out[i] = ggo_sample_one(beta, alpha, seed, tensor_id, index0 + (uint64_t)i, &att);
        if (attempts) attempts[i] = (uint8_t)att;
    }
}

/* Standard-normal and Gamma(a',1) intermediates of attempt 0 only, exposed so
 * that the tests can pin Box-Muller and the acceptance rule separately. */
void ggo_sample_debug(double beta, uint64_t seed, uint32_t tensor_id, uint64_t index,
                      uint32_t attempt, double *z_out, double *lhs_out, double *rhs_out)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t ctr[4] = { (uint32_t)index, (uint32_t)(index >> 32), attempt, tensor_id };
    uint32_t r[4];
    ggo_philox4x32_10(ctr, key, r);
    double a = 1.0 / beta;
    double a1 = a >= 1.0 ? a : a + 1.0;
    double d = a1 - 1.0 / 3.0;
    double c = 1.0 / sqrt(9.0 * d);
    double z = sqrt(-2.0 * log(ggo_u01(r[0]))) * cos(GGO_TWO_PI * ggo_u01(r[1]));
    double w = 1.0 + c * z;
    double v = w * w * w;
    *z_out = z;
    *lhs_out = log(ggo_u01(r[2]));
    *rhs_out = w > 0.0 ? 0.5 * z * z + d * (1.0 - v + log(v)) : -INFINITY;
}

/* ------------------------------------------- Exponential-Golomb rate (Eq. 6-7) */

/* Eq. 6: the signed symbol to the unsigned one that is coded: q < 0 -> -2q, 0 -> 0, q > 0 -> 2q - 1. */
uint64_t ggo_map(int64_t q)
{
    if (q < 0) return (uint64_t)(-2 * q);
    if (q == 0) return 0;
    return (uint64_t)(2 * q - 1);
}

/* Length in bits of the k-th order Exponential-Golomb code of m >= 0:
 * 2 floor(log2(m + 2^k)) - k + 1.  (Eq. 7 prints this with its floor written as a straight-through
 * operator and the "- k + 1" outside the mean; read as the standard code length.)  The floor of
 * the logarithm is the position of the highest set bit, found by shifting. */
int32_t ggo_eg_length(uint64_t m, int32_t k)
{
    uint64_t v = m + ((uint64_t)1 << k);
    int32_t fl = -1;
    while (v) { v >>= 1; ++fl; }
    return 2 * fl - k + 1;
}

/* Eq. 7 for one tensor, element by element: quantise (the fp32-defined floor quantiser above, with
 * the clamp), map, take the code length, average.  n = 0 gives 0. */
double ggo_eg_rate(const float *x, int64_t n, float step, int32_t qmin, int32_t qmax, int32_t k)
{
    const float inv = (float)(1.0 / (double)step);
    long double bits = 0.0L;
    int64_t counted = 0;
    for (int64_t i = 0; i < n; ++i) {
        const float t = x[i] * inv;
        double f = floor((double)t);
        if (isnan(f)) continue;
        int64_t q;
        if (f < (double)qmin) q = qmin; else if (f > (double)qmax) q = qmax; else q = (int64_t)f;
        bits += (long double)ggo_eg_length(ggo_map(q), k);
        ++counted;
    }
    return counted ? (double)(bits / (long double)counted) : 0.0;
}

/* The same rate from a count table (bin b holds symbol qmin + b). */
double ggo_eg_rate_hist(const uint64_t *hist, int64_t n_bins, int32_t qmin, int32_t k)
{
    long double bits = 0.0L, total = 0.0L;
    for (int64_t b = 0; b < n_bins; ++b) {
        if (!hist[b]) continue;
        bits += (long double)hist[b] * (long double)ggo_eg_length(ggo_map((int64_t)qmin + b), k);
        total += (long double)hist[b];
    }
    return total > 0.0L ? (double)(bits / total) : 0.0;
}

/* Gradient of lambda * R with respect to the elements, the paper's
 *     dR/dG = 2^(n+2) / (N ln 2) * Sign(G) / Map(Quant(G))
 * with 2^n = 1/step, N the element count, and the denominator read as m + 2^k (the derivative of
 * 2 log2(m + 2^k); the printed form leaves 2^k out and divides by zero at m = 0):
 *     g_i = lambda * 4 / (step N ln 2) * sign(x_i) / (Map(q_i) + 2^k),   sign(0) = 0.
 * The scaling 1/step is the quantiser's fp32 inv, so that both sides use the same number. */
void ggo_eg_rate_grad(const float *x, int64_t n, float step, int32_t qmin, int32_t qmax, int32_t k,
                      double lambda, double *grad)
{
    const float inv = (float)(1.0 / (double)step);
    const double c = n > 0 ? lambda * 4.0 * (double)inv / ((double)n * log(2.0)) : 0.0;
    for (int64_t i = 0; i < n; ++i) {
        const float t = x[i] * inv;
        double f = floor((double)t);
        double g = 0.0;
        if (!isnan(f) && x[i] != 0.0f) {
            int64_t q;
            if (f < (double)qmin) q = qmin; else if (f > (double)qmax) q = qmax; else q = (int64_t)f;
            g = c / (double)(ggo_map(q) + ((uint64_t)1 << k));
            if (x[i] < 0.0f) g = -g;
        }
        grad[i] = g;
    }
}

/* ------------------------------------------------ Huffman and fixed-length bits */

/* Average length in bits of a Huffman code for the counts, by the textbook construction written out:
 * every occupied bin is a leaf; while more than one root is left, the two lightest roots (found by a
 * scan of the whole list) become the children of a new root whose weight is their sum; the code
 * length of a symbol is the depth of its leaf; the average is sum(count * length) / sum(count).
 * One occupied bin gives 0 bits.  Quadratic in the number of occupied bins: a checker, not a coder.
 * work: scratch of 2 * n_bins uint64 (node weights); parent links and root marks are allocated here. */
double ggo_huffman_bits(const uint64_t *hist, int64_t n_bins, uint64_t *work)
{
    int64_t n = 0;
    for (int64_t b = 0; b < n_bins; ++b) if (hist[b]) work[n++] = hist[b];
    if (n <= 1) return 0.0;
    int64_t *parent = (int64_t *)malloc(sizeof(int64_t) * (size_t)(2 * n));
    char *is_root = (char *)malloc((size_t)(2 * n));
    if (!parent || !is_root) { free(parent); free(is_root); return NAN; }
    for (int64_t i = 0; i < n; ++i) { parent[i] = -1; is_root[i] = 1; }
    int64_t nodes = n;
    for (int64_t roots = n; roots > 1; --roots) {
        int64_t first = -1, second = -1;       /* the lightest and the next lightest root */
        for (int64_t i = 0; i < nodes; ++i) {
            if (!is_root[i]) continue;
            if (first < 0 || work[i] < work[first]) { second = first; first = i; }
            else if (second < 0 || work[i] < work[second]) second = i;
        }
        work[nodes] = work[first] + work[second];
        parent[nodes] = -1; is_root[nodes] = 1;
        parent[first] = nodes; parent[second] = nodes;
        is_root[first] = 0; is_root[second] = 0;
        ++nodes;
    }
    long double bits = 0.0L, total = 0.0L;
    for (int64_t leaf = 0; leaf < n; ++leaf) {
        int64_t depth = 0;
        for (int64_t v = leaf; parent[v] >= 0; v = parent[v]) ++depth;
        bits += (long double)work[leaf] * (long double)depth;
        total += (long double)work[leaf];
    }
    free(parent); free(is_root);
    return (double)(bits / total);
}

/* Bits of a fixed-length code over the occupied symbol range: ceil(log2(max - min + 1)); an empty
 * table or a single symbol gives 0.  (The paper reports FL without defining it; its values are
 * whole numbers of bits.) */
int32_t ggo_fixed_length_bits(const uint64_t *hist, int64_t n_bins)
{
    int64_t lo = -1, hi = -1;
    for (int64_t b = 0; b < n_bins; ++b) if (hist[b]) { if (lo < 0) lo = b; hi = b; }
    if (lo < 0) return 0;
    uint64_t span = (uint64_t)(hi - lo);   /* symbols - 1 */
    int32_t bits = 0;
    while (span) { span >>= 1; ++bits; }
    return bits;
}

/* --------------------------------------------------- GCT elementwise update (Algorithm 2) */

/* One step of gradient constrained training for one tensor, the three elementwise lines of
 * Algorithm 2 in their printed order, in fp64:
 *     h_i    = ( -(1/eta) g_i / (ghat_prev_i + eps) + 1/eta ) * [t >= 2]
 *     ghat_i = g_i + lambda * dR/dg_i * h_i        (dR/dg: ggo_eg_rate_grad with lambda = 1)
 *     w_i   <- w_i - eta * ghat_i
 * eps is added to the signed previous gradient exactly as printed.  ghat_out is what the next step
 * needs as ghat_prev. */
void ggo_gct_step(const float *g, const double *ghat_prev, const double *w, int64_t n, float step,
                  int32_t qmin, int32_t qmax, int32_t k, double eta, double lambda, double eps,
                  int64_t t, double *drdg_work, double *ghat_out, double *w_out)
{
    ggo_eg_rate_grad(g, n, step, qmin, qmax, k, 1.0, drdg_work);
    for (int64_t i = 0; i < n; ++i) {
        double h = 0.0;
        if (t >= 2) h = -(1.0 / eta) * (double)g[i] / (ghat_prev[i] + eps) + 1.0 / eta;
        const double gh = (double)g[i] + lambda * drdg_work[i] * h;
        ghat_out[i] = gh;
        w_out[i] = w[i] - eta * gh;
    }
}
