// Moment-ratio inversion from a table (shared by the per-segment fit kernels and the short-segment
// kernel), and the short exponential the gradient tables are built with.
//
// The table holds, on kSeedCells cells of a uniform grid of u = ln(beta) over
// [ln GG_BETA_LO, ln GG_BETA_HI], the two smooth functions the fit needs:
//     Y(u) = ln rho(beta) = 2 lgamma(2/beta) - lgamma(1/beta) - lgamma(3/beta)    (increasing in u)
//     Z(u) = ln(alpha / sigma) = (lgamma(1/beta) - lgamma(3/beta)) / 2             (Eq. 2)
// Given ln r, the cell with Y[i] <= ln r < Y[i+1] is found by bisection of the table, and u is the
// root of the cubic through the four nodes around the cell (Newton from the linear guess).  With
// 2048 cells the cubic is within 1e-11 of Y and Z over the whole range, so beta and alpha come out
// to about 1e-10 relative without a single lgamma at fit time.
#pragma once
#include "gg_internal.h"

namespace gg {

// Values and derivatives of the cubic Lagrange basis on the nodes -1, 0, 1, 2.
__device__ __forceinline__ void cubic_basis(double t, double (&w)[4], double (&d)[4])
{
    const double a = t + 1.0, b = t, c = t - 1.0, e = t - 2.0;
    w[0] = -b * c * e * (1.0 / 6.0);
    w[1] = a * c * e * 0.5;
    w[2] = -a * b * e * 0.5;
    w[3] = a * b * c * (1.0 / 6.0);
    d[0] = -(c * e + b * e + b * c) * (1.0 / 6.0);
    d[1] = (c * e + a * e + a * c) * 0.5;
    d[2] = -(b * e + a * e + a * b) * 0.5;
    d[3] = (b * c + a * c + a * b) * (1.0 / 6.0);
}

// table: Y[0 .. kSeedCells] followed by Z[0 .. kSeedCells].  log_r must lie strictly between Y[0] and
// Y[kSeedCells].  Returns beta and writes ln(alpha / sigma).
// WARP: all 32 lanes of the warp call with the same log_r; the cell is then found in three rounds of 32
// look-ups side by side instead of eleven one after the other.
template <bool WARP = false>
__device__ __forceinline__ double invert_ratio_table(double log_r, const double *table, double *ln_alpha_over_sigma)
{
    const double *Y = table, *Z = table + (kSeedCells + 1);
    int i0 = 0;                             // Y[i0] <= log_r < Y[i0 + 1]
    if constexpr (WARP) {
        static_assert(kSeedCells == 2048, "two rounds of 32 and one of 2");
        const int lane = threadIdx.x & 31;
        // nodes 64 l, then 2 l inside the block of 64, then the odd node: each ballot counts the nodes <= log_r
        i0 = 64 * (__popc(__ballot_sync(0xFFFFFFFFu, __ldg(Y + 64 * lane) <= log_r)) - 1);
        i0 += 2 * (__popc(__ballot_sync(0xFFFFFFFFu, __ldg(Y + i0 + 2 * lane) <= log_r)) - 1);
        if (__ldg(Y + i0 + 1) <= log_r) i0 += 1;
    } else {
        int i1 = kSeedCells;
        while (i1 - i0 > 1) {
            const int m = (i0 + i1) >> 1;
            if (__ldg(Y + m) <= log_r) i0 = m; else i1 = m;
        }
    }
    const int j = max(0, min(kSeedCells - 3, i0 - 1));     // first node of the four-point stencil
    const double y0 = __ldg(Y + j), y1 = __ldg(Y + j + 1), y2 = __ldg(Y + j + 2), y3 = __ldg(Y + j + 3);
    const double ya = __ldg(Y + i0), yb = __ldg(Y + i0 + 1);
    double t = (double)(i0 - j - 1) + (log_r - ya) / (yb - ya);
    double w[4], d[4];
    // (from the linear guess one Newton step leaves 3e-12 in ln beta, two leave 2e-14: below the cubic's own 1e-11)
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        cubic_basis(t, w, d);
        const double f = w[0] * y0 + w[1] * y1 + w[2] * y2 + w[3] * y3 - log_r;
        const double fp = d[0] * y0 + d[1] * y1 + d[2] * y2 + d[3] * y3;
        t -= f / fp;
    }
    cubic_basis(t, w, d);
    *ln_alpha_over_sigma = w[0] * __ldg(Z + j) + w[1] * __ldg(Z + j + 1) + w[2] * __ldg(Z + j + 2) + w[3] * __ldg(Z + j + 3);
    const double u0 = log(GG_BETA_LO), h = (log(GG_BETA_HI) - log(GG_BETA_LO)) / (double)kSeedCells;
    return exp(u0 + h * ((double)(j + 1) + t));
}

// The fit of one segment from its sums: beta from the moment ratio, alpha from Eq. 2 with
// sigma^2 = sum_sq / len.  Returns the GG_FLAG_* bits of the fit (degenerate, clamped).
__device__ __forceinline__ uint32_t fit_from_sums(double s1, double s2, int64_t len, const double *table, double *beta,
                                                  double *alpha)
{
    *beta = 0.0;
    *alpha = 0.0;
    if (len <= 0 || !(s2 > 0.0)) return GG_FLAG_DEGENERATE;
    const double m1 = s1 / (double)len, m2 = s2 / (double)len;
    const double log_r = log(m1 * m1 / m2);
    uint32_t flags = 0u;
    double lnz;
    if (log_r <= __ldg(table)) {
        *beta = GG_BETA_LO;
        lnz = __ldg(table + kSeedCells + 1);
        flags = GG_FLAG_BETA_CLAMPED_LO;
    } else if (log_r >= __ldg(table + kSeedCells)) {
        *beta = GG_BETA_HI;
        lnz = __ldg(table + 2 * kSeedCells + 1);
        flags = GG_FLAG_BETA_CLAMPED_HI;
    } else {
        *beta = invert_ratio_table(log_r, table, &lnz);
    }
    *alpha = sqrt(m2) * exp(lnz);
    return flags;
}

// Flat-topped data make the fit ill-conditioned: d ln(beta) / d ln(rho) grows from 4 at beta = 2 to 150 at beta = 20, so
// above rho(4) = 1/sqrt(2) the last bits of the fp32 run sums that the sweeps feed into their fp64 partials (about 1e-7
// relative for a segment of a single run) would show in the fifth digit of beta.  In a long segment those roundings
// average out; for a short one the warp that fits takes the two sums again in fp64 straight from the elements (at most
// kCarefulLen of them: a microsecond or two, and rare), in a fixed order, non-finite entries left out as everywhere.
constexpr int64_t kCarefulLen = 8192;
constexpr double kCarefulLogRatio = -0.34657359027997264;      // ln rho(4) = -ln(2) / 2

// WARP: all 32 lanes call with the same arguments and end with the same sums.
__device__ __forceinline__ void careful_sums(const void *ptr, int in_dtype, int64_t len, int lane, double &s1, double &s2)
{
    double t1 = 0.0, t2 = 0.0;
    if (in_dtype == GG_F32) {
        const float *x = static_cast<const float *>(ptr);
        for (int64_t i = lane; i < len; i += 32) {
            const uint32_t ab = __float_as_uint(__ldg(x + i)) & 0x7FFFFFFFu;
            if (ab < 0x7F800000u) { const double ax = (double)__uint_as_float(ab); t1 += ax; t2 = fma(ax, ax, t2); }
        }
    } else {
        const uint16_t *x = static_cast<const uint16_t *>(ptr);
        for (int64_t i = lane; i < len; i += 32) {
            const uint32_t h = (uint32_t)__ldg(x + i) & 0x7FFFu;
            if (h < 0x7F80u) { const double ax = (double)__uint_as_float(h << 16); t1 += ax; t2 = fma(ax, ax, t2); }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        t1 += __shfl_xor_sync(0xFFFFFFFFu, t1, o);
        t2 += __shfl_xor_sync(0xFFFFFFFFu, t2, o);
    }
    s1 = t1;
    s2 = t2;
}

// ln of rho(beta) = Gamma(2/beta)^2 / (Gamma(1/beta) Gamma(3/beta)), the ratio (E|x|)^2 / E[x^2]
// of the density of Eq. 1; increasing in beta from 0 to 3/4.
__device__ __forceinline__ double log_rho(double beta)
{
    return 2.0 * lgamma(2.0 / beta) - lgamma(1.0 / beta) - lgamma(3.0 / beta);
}

// The fit of segment s from its reduced sums and extremes, and every per-segment output of the fit step
// (parameters, sums, count, flags, the quantiser step taken from alpha, the standard deviation for the sweep
// that follows).  WARP: all 32 lanes of a warp call with the same arguments; lane 0 writes.  Without a fit table
// (a.seed null) the root is found by 33-section search on ln(beta): each round the 32 lanes evaluate log_rho at
// the interior points of the bracket and a ballot picks the sub-interval with the sign change.
// The results every lane holds on return: the parameters and the quantiser step of the segment.
struct FitResult {
    double beta, alpha;
    float step;
};

__device__ __forceinline__ FitResult fit_finish(const FitArgs &a, int s, int lane, double s1, double s2, uint32_t bad, float xmin,
                                                float xmax)
{
    constexpr unsigned kFull = 0xFFFFFFFFu;
    const int64_t len = a.map.seg_len[s];

    uint32_t flags = bad ? GG_FLAG_NONFINITE : 0u;
    double beta = 0.0, alpha = 0.0;
    if (len <= 0 || !(s2 > 0.0)) {
        flags |= GG_FLAG_DEGENERATE;
    } else {
        double m1 = s1 / (double)len, m2 = s2 / (double)len;
        double log_r = log(m1 * m1 / m2);
        if (log_r > kCarefulLogRatio && len <= kCarefulLen && a.in_dtype_plus1 != 0) {
            careful_sums(a.map.seg_ptr[s], a.in_dtype_plus1 - 1, len, lane, s1, s2);
            m1 = s1 / (double)len;
            m2 = s2 / (double)len;
            log_r = log(m1 * m1 / m2);
        }
        if (a.seed != nullptr) {
            // table look-up and cubic interpolation (no lgamma at fit time)
            double lnz;
            if (log_r <= __ldg(a.seed)) {
                beta = GG_BETA_LO;
                lnz = __ldg(a.seed + kSeedCells + 1);
                flags |= GG_FLAG_BETA_CLAMPED_LO;
            } else if (log_r >= __ldg(a.seed + kSeedCells)) {
                beta = GG_BETA_HI;
                lnz = __ldg(a.seed + 2 * kSeedCells + 1);
                flags |= GG_FLAG_BETA_CLAMPED_HI;
            } else {
                beta = invert_ratio_table<true>(log_r, a.seed, &lnz);      // (every lane is here with the same log_r)
            }
            alpha = sqrt(m2) * exp(lnz);
        } else {
        if (log_r <= log_rho(GG_BETA_LO)) {
            beta = GG_BETA_LO;
            flags |= GG_FLAG_BETA_CLAMPED_LO;
        } else if (log_r >= log_rho(GG_BETA_HI)) {
            beta = GG_BETA_HI;
            flags |= GG_FLAG_BETA_CLAMPED_HI;
        } else {
            double lo = log(GG_BETA_LO), hi = log(GG_BETA_HI);
            for (int round = 0; round < 12 && hi - lo > 4e-15; ++round) {
                const double w = (hi - lo) * (1.0 / 33.0);
                const double ti = lo + w * (double)(lane + 1);
                const bool below = log_rho(exp(ti)) < log_r;
                const int k = __popc(__ballot_sync(kFull, below));   // points 1..k lie below the root
                hi = lo + w * (double)(k + 1);
                lo = lo + w * (double)k;
            }
            beta = exp(0.5 * (lo + hi));
        }
        alpha = sqrt(m2) * exp(0.5 * (lgamma(1.0 / beta) - lgamma(3.0 / beta)));
        }
    }
    const float step = a.step_from_alpha ? (float)(alpha * a.step_scale) : (a.step ? a.step[s] : 0.0f);
    if (lane == 0) {
        a.beta[s] = beta;
        a.alpha[s] = alpha;
        if (a.sum_abs) a.sum_abs[s] = s1;
        if (a.sum_sq) a.sum_sq[s] = s2;
        if (a.count) a.count[s] = len;
        if (a.step_from_alpha && a.step_out) a.step_out[s] = step;
        if (a.hist_on && xmin <= xmax) {
            // the quantiser is monotone in x, so a symbol clamps iff one of the extremes does
            const float inv = (float)(1.0 / (double)step);
            const float tlo = __fmul_rn(xmin, inv), thi = __fmul_rn(xmax, inv);
            if ((double)floorf(tlo) < (double)a.qmin || (double)floorf(thi) > (double)a.qmax)
                flags |= GG_FLAG_CLAMPED_SYMBOLS;
        }
        if (a.flags) a.flags[s] = flags;
        if (a.sd_out) a.sd_out[s] = (len > 0 && s2 > 0.0) ? sqrt(s2 / (double)len) : 0.0;
    }
    return FitResult{beta, alpha, step};
}

// 2^t for |t| < 1000 within 1e-11 relative: table entries are rounded to fp32 afterwards.
__device__ __forceinline__ double exp2_short(double t)
{
    const double n = rint(t);
    const double f = (t - n) * 0.69314718055994531;      // |f| <= 0.3466
    double p = 1.0 / 3628800.0;                           // Taylor series of e^f to degree 10
    p = fma(p, f, 1.0 / 362880.0);
    p = fma(p, f, 1.0 / 40320.0);
    p = fma(p, f, 1.0 / 5040.0);
    p = fma(p, f, 1.0 / 720.0);
    p = fma(p, f, 1.0 / 120.0);
    p = fma(p, f, 1.0 / 24.0);
    p = fma(p, f, 1.0 / 6.0);
    p = fma(p, f, 0.5);
    p = fma(p, f, 1.0);
    p = fma(p, f, 1.0);
    return p * __hiloint2double(((int)n + 1023) << 20, 0);
}

}  // namespace gg
