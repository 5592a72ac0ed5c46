// The GG pass over the COLUMNS of a row-major bf16 matrix (one generalized Gaussian per channel).
//
// A column is a strided segment, so the kernels are tiled the other way round from the contiguous
// path: a strip of 64 neighbouring columns is 128 contiguous bytes of every row, a warp reads one
// such row piece per load (lane l holds columns 2l and 2l+1 as one 32-bit word) and walks down the
// rows, so every thread accumulates the sums of its own two columns and no transposition happens.
//   chan_moments_kernel   one CTA per (strip, block of 256 rows): sum |x|, sum x^2, non-finite
//                         count, min, max per column, written per row block
//   chan_fit_kernel       one thread per column: adds the row blocks in order, inverts the moment
//                         ratio from the fit table, derives the constants of the gradient
//   chan_tail_kernel      one CTA per (strip, slice of rows): builds the per-column gradient tables
//                         |g| = A_c[e] * B_c[j] (e exponent field, j mantissa bits of the bf16
//                         pattern; the lane owns its columns, so lane l reads word l of a table
//                         row and no look-up ever meets a bank conflict), then streams its rows:
//                         gradient, penalty partial per column, symbol counts in shared memory
//   chan_penalty_kernel   one thread per column: adds the slices in order, divides by beta
// A is kept for a window of 64 exponents below the largest magnitude of the strip; every exponent
// outside it, zero/subnormal/inf/nan and far binades read a NaN marker, the NaN reaches the
// column's penalty partial of the current block of rows, and the range check of that partial
// sends the block's column to an exact fp64 path.  Exact zeros are common in activations and are
// selected to a zero gradient without the exact path.
#include <cuda_bf16.h>
#include <float.h>

#include "gg_fit_table.cuh"
#include "gg_internal.h"

namespace gg {
namespace {

constexpr int kMomThreads = 256;
constexpr int kMomWarps = kMomThreads / 32;
constexpr int kU = 8;                      // rows in flight per thread

constexpr int kTailThreads = 512;
constexpr int kTailWarps = kTailThreads / 32;
constexpr int kCtasPerSm = 2;
constexpr int kAWin = 64;                  // exponents covered by the A table (row kAWin: the marker)
constexpr int kSymWin = 4096;              // symbols counted in shared memory: [-2048, 2048) cut to [qmin, qmax]
constexpr uint32_t kMagicBits = 0x4B400000u;   // 1.5 * 2^23: floor(t) = bits(t +rd magic) - bits(magic)

// The 32-bit word of columns (2 lane, 2 lane + 1) of one row; missing columns read as zero.
__device__ __forceinline__ uint32_t load_pair(const uint16_t *row, bool vec, bool ok0, bool ok1)
{
    if (vec) return ok0 ? __ldg(reinterpret_cast<const uint32_t *>(row)) : 0u;   // (vec: cols is even, ok0 == ok1)
    uint32_t w = 0;
    if (ok0) w = (uint32_t)__ldg(row);
    if (ok1) w |= (uint32_t)__ldg(row + 1) << 16;
    return w;
}

// One column's share of a block of rows, in fp64, non-finite entries left out (used when the fp32
// partials of the block left the fp32 range).
__device__ __noinline__ void moments_careful(const uint32_t (&w)[kU], int half, double &s1, double &s2)
{
    for (int u = 0; u < kU; ++u) {
        const uint32_t h = (half ? (w[u] >> 16) : w[u]) & 0x7FFFu;
        if (h < 0x7F80u) {
            const double ax = (double)__uint_as_float(h << 16);
            s1 += ax;
            s2 += ax * ax;
        }
    }
}

__global__ void __launch_bounds__(kMomThreads) chan_moments_kernel(const ChanArgs a)
{
    __shared__ double red1[kMomWarps][kChanStrip], red2[kMomWarps][kChanStrip];
    __shared__ uint32_t redb[kMomWarps][kChanStrip];
    __shared__ float redmn[kMomWarps][kChanStrip], redmx[kMomWarps][kChanStrip];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kChanStrip + 2 * lane;
    const int64_t r_begin = (int64_t)blockIdx.y * kChanMomRows;
    const int64_t r_end = min(a.rows, r_begin + kChanMomRows);
    const bool ok0 = c0 < a.cols, ok1 = c0 + 1 < a.cols;
    const bool vec = ((reinterpret_cast<uintptr_t>(a.x) & 3u) == 0) && ((a.ld & 1) == 0) && ((a.cols & 1) == 0);
    const uint16_t *col = a.x + c0;

    double s1[2] = {0.0, 0.0}, s2[2] = {0.0, 0.0};
    uint32_t bad[2] = {0u, 0u};
    float mn[2] = {INFINITY, INFINITY}, mx[2] = {-INFINITY, -INFINITY};
    for (int64_t r = r_begin + warp; r < r_end; r += (int64_t)kMomWarps * kU) {
        uint32_t w[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int64_t ru = r + (int64_t)u * kMomWarps;
            w[u] = ru < r_end ? load_pair(col + ru * a.ld, vec, ok0, ok1) : 0u;
        }
        float m1[2] = {0.0f, 0.0f}, m2[2] = {0.0f, 0.0f};
#pragma unroll
        for (int u = 0; u < kU; ++u) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const uint32_t xb = k ? (w[u] & 0xFFFF0000u) : (w[u] << 16);
                const float ax = __uint_as_float(xb & 0x7FFFFFFFu);
                m1[k] += ax;
                m2[k] = fmaf(ax, ax, m2[k]);
                bad[k] += (xb & 0x7FFFFFFFu) >= 0x7F800000u ? 1u : 0u;
                mn[k] = fminf(mn[k], __uint_as_float(xb));      // fminf / fmaxf return the non-NaN operand
                mx[k] = fmaxf(mx[k], __uint_as_float(xb));
            }
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            // (rows past the end and missing columns were read as zero: they add nothing; the extremes are
            // corrected below)
            if (run_sums_exact_enough(m1[k], m2[k])) { s1[k] += (double)m1[k]; s2[k] += (double)m2[k]; }
            else moments_careful(w, k, s1[k], s2[k]);     // inf, nan, or squares outside the fp32 range
        }
    }
    // Rows past the end and missing columns entered the extremes as zeros.  Only the last row block and
    // the last strip can have them: there the extremes are taken again over the real entries alone.
    if (r_end - r_begin < kChanMomRows || !ok0 || !ok1) {
        for (int k = 0; k < 2; ++k) { mn[k] = INFINITY; mx[k] = -INFINITY; }
        for (int64_t r = r_begin + warp; r < r_end; r += kMomWarps) {
            const uint32_t w = load_pair(col + r * a.ld, vec, ok0, ok1);
            const float v0 = __uint_as_float(w << 16), v1 = __uint_as_float(w & 0xFFFF0000u);
            if (ok0) { mn[0] = fminf(mn[0], v0); mx[0] = fmaxf(mx[0], v0); }
            if (ok1) { mn[1] = fminf(mn[1], v1); mx[1] = fmaxf(mx[1], v1); }
        }
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        red1[warp][2 * lane + k] = s1[k];
        red2[warp][2 * lane + k] = s2[k];
        redb[warp][2 * lane + k] = bad[k];
        redmn[warp][2 * lane + k] = mn[k];
        redmx[warp][2 * lane + k] = mx[k];
    }
    __syncthreads();
    if (threadIdx.x < kChanStrip) {
        const int64_t c = (int64_t)blockIdx.x * kChanStrip + threadIdx.x;
        if (c < a.cols) {
            double r1 = 0.0, r2 = 0.0;
            uint32_t rb = 0;
            float rmn = INFINITY, rmx = -INFINITY;
            for (int w = 0; w < kMomWarps; ++w) {     // fixed order
                r1 += red1[w][threadIdx.x]; r2 += red2[w][threadIdx.x]; rb += redb[w][threadIdx.x];
                rmn = fminf(rmn, redmn[w][threadIdx.x]); rmx = fmaxf(rmx, redmx[w][threadIdx.x]);
            }
            const int64_t o = (int64_t)blockIdx.y * a.cols + c;
            a.s1[o] = r1; a.s2[o] = r2; a.bad[o] = rb; a.xmin[o] = rmn; a.xmax[o] = rmx;
        }
    }
}

// One thread per column: the row blocks in order, the fit, the clamp flag, the gradient constants.
__global__ void __launch_bounds__(128) chan_fit_kernel(const ChanArgs a)
{
    const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= a.cols) return;
    double s1 = 0.0, s2 = 0.0;
    uint32_t bad = 0;
    float xmin = INFINITY, xmax = -INFINITY;
    for (int k = 0; k < a.n_mom_blocks; ++k) {
        const int64_t o = (int64_t)k * a.cols + c;
        s1 += a.s1[o]; s2 += a.s2[o]; bad += a.bad[o];
        xmin = fminf(xmin, a.xmin[o]); xmax = fmaxf(xmax, a.xmax[o]);
    }
    double beta, alpha;
    uint32_t flags = fit_from_sums(s1, s2, a.rows, a.seed, &beta, &alpha) | (bad ? GG_FLAG_NONFINITE : 0u);
    if (a.do_hist && xmin <= xmax) {
        // the quantiser is monotone in x, so a symbol clamps iff one of the extremes does
        const float inv = (float)(1.0 / (double)a.step);
        const float tlo = __fmul_rn(xmin, inv), thi = __fmul_rn(xmax, inv);
        if ((double)floorf(tlo) < (double)a.qmin || (double)floorf(thi) > (double)a.qmax) flags |= GG_FLAG_CLAMPED_SYMBOLS;
    }
    a.beta[c] = beta;
    a.alpha[c] = alpha;
    if (a.sum_abs) a.sum_abs[c] = s1;
    if (a.sum_sq) a.sum_sq[c] = s2;
    if (a.count) a.count[c] = a.rows;
    if (a.flags) a.flags[c] = flags;
    const bool active = (beta > 0.0) && (alpha > 0.0) && (a.lambda != 0.0) && (a.lambda == a.lambda);
    a.L[c] = active ? log2(fabs(a.lambda) * beta) - beta * log2(alpha) : __longlong_as_double(0x7FF8000000000000ll);
    a.b[c] = beta - 1.0;
    // the largest finite magnitude places the exponent window of the strip's A tables
    float am = 0.0f;
    if (xmin <= xmax) {
        const float lo = fabsf(xmin), hi = fabsf(xmax);
        am = fmaxf(lo <= FLT_MAX ? lo : FLT_MAX, hi <= FLT_MAX ? hi : FLT_MAX);
    }
    a.amax[c] = am;
}

__global__ void __launch_bounds__(128) chan_penalty_kernel(const ChanArgs a)
{
    const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= a.cols) return;
    double p = 0.0;
    for (int k = 0; k < a.n_slices; ++k) p += a.pen[(int64_t)k * a.cols + c];
    const double beta = a.beta[c];
    // sum |x| |g| = |lambda| beta sum (|x|/alpha)^beta; the penalty carries lambda's sign
    a.penalty[c] = beta > 0.0 ? (a.lambda < 0.0 ? -p : p) / beta : 0.0;
}

// ------------------------------------------------------------------------------------ second kernel

struct TailSmem {
    float a1[2][kAWin + 1][32];       // [k][e - e_lo][lane]: A of column 2 lane + k; row kAWin: the marker
    float bt[2][128][32];             // [k][j][lane]: B of column 2 lane + k
    uint32_t cnt[kSymWin + 2];        // cell 0 and the last: sentinels of the two tails
    double red[kTailWarps][kChanStrip];
    double colL[kChanStrip], colb[kChanStrip];
    double lg[128];                   // log2(1 + j/128)
    uint32_t clampc[2];
    int e_top;
};

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

// Exact gradient magnitude (with lambda's sign through `flip`) of a 15-bit magnitude pattern.
__device__ __noinline__ float chan_grad_exact(uint32_t mag, double L, double b, uint32_t flip)
{
    const float ax = __uint_as_float(mag << 16);
    if (!(L == L) || ax == 0.0f) return 0.0f;
    const float v = (float)exp2(L + b * log2((double)ax));
    return __uint_as_float(__float_as_uint(v) ^ flip);
}

// fp64 penalty terms |x| |g| of one column over a block of rows.
__device__ __noinline__ double chan_pen_exact(const uint32_t (&w)[kU], int half, double L, double b)
{
    if (!(L == L)) return 0.0;
    double dp = 0.0;
    for (int u = 0; u < kU; ++u) {
        const uint32_t h = (half ? (w[u] >> 16) : w[u]) & 0x7FFFu;
        const double ax = (double)__uint_as_float(h << 16);
        if (ax != 0.0) dp += ax * exp2(L + b * log2(ax));
    }
    return dp;
}

// Quantises one value and counts its symbol: the shared window when in reach, else global memory.
__device__ __noinline__ void chan_count_slow(float x, float inv, int32_t qmin, int32_t qmax, int32_t wlo, int32_t whi,
                                             TailSmem &sm, unsigned long long *hist)
{
    const float t = __fmul_rn(x, inv);
    if (t == t) {                                  // NaN is skipped
        int q = __float2int_rd(t);                 // floor, saturating
        if (q < qmin) { q = qmin; atomicAdd(&sm.clampc[0], 1u); }
        else if (q > qmax) { q = qmax; atomicAdd(&sm.clampc[1], 1u); }
        if (q >= wlo && q < whi) atomicAdd(&sm.cnt[q - wlo + 1], 1u);
        else atomicAdd(&hist[q - qmin], 1ull);
    }
}

__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

__device__ __forceinline__ void red_inc(uint32_t addr)
{
    asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}

// Per-thread constants of the element path.
struct ChanLane {
    uint32_t a_addr[2], b_addr[2];   // shared-memory addresses of this lane's word in row 0 of its tables
    uint32_t e_lo;                   // exponent field of row 0 of the A tables
    uint32_t cnt_off;                // cell of a value = bits(floor(t) + magic) * 4 + cnt_off (mod 2^32)
    float inv, t_lo, t_hi;           // quantiser scale; t is clamped to [t_lo, t_hi] so that its floor is a cell
};

// One element (HALF 0: the low half of w, the lane's even column).  Branch free.
template <bool GRAD, bool HIST, int HALF>
__device__ __forceinline__ float chan_elem(uint32_t w, bool counted, const ChanLane &ln, float &mp, uint32_t &anyc)
{
    const uint32_t xb = HALF ? (w & 0xFFFF0000u) : (w << 16);
    float g = 0.0f;
    if constexpr (GRAD) {
        const uint32_t e = HALF ? (w >> 23) & 0xFFu : (w >> 7) & 0xFFu;
        const uint32_t j = HALF ? (w >> 16) & 127u : w & 127u;
        const uint32_t i = min(e - ln.e_lo, (uint32_t)kAWin);       // below the window wraps around to the marker too
        float ga = lds_f32(ln.a_addr[HALF] + i * 128u) * lds_f32(ln.b_addr[HALF] + j * 128u);
        ga = (xb << 1) == 0u ? 0.0f : ga;                            // g(0) = 0 for every shape
        mp = fmaf(fabsf(__uint_as_float(xb)), fabsf(ga), mp);
        g = __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));   // the table carries lambda's sign
    }
    if constexpr (HIST) {
        if (counted) {
            const float t = __fmul_rn(__uint_as_float(xb), ln.inv);
            anyc = max(anyc, __float_as_uint(t) & 0x7FFFFFFFu);
            // outside the window (and nan, which fmaxf replaces by the lower bound) the floor lands on a sentinel
            const float tc = fminf(fmaxf(t, ln.t_lo), ln.t_hi);
            // |tc| < 2^22: the sum lies in [2^23, 2^24) where floats are the integers, so rounding down gives floor
            const uint32_t fb = __float_as_uint(__fadd_rd(tc, __uint_as_float(kMagicBits)));
            red_inc(fb * 4u + ln.cnt_off);
        }
    }
    return g;
}

template <typename TG>
__device__ __forceinline__ void store_pair(TG *p, float g0, float g1, bool vec, bool ok0, bool ok1, bool accumulate)
{
    if constexpr (sizeof(TG) == 4) {
        if (vec) {
            if (!ok0) return;
            float2 *q = reinterpret_cast<float2 *>(p);
            if (accumulate) { const float2 old = *q; g0 += old.x; g1 += old.y; }
            __stcs(q, make_float2(g0, g1));
        } else {
            if (ok0) p[0] = accumulate ? p[0] + g0 : g0;
            if (ok1) p[1] = accumulate ? p[1] + g1 : g1;
        }
    } else {
        if (vec) {
            if (!ok0) return;
            uint32_t *q = reinterpret_cast<uint32_t *>(p);
            if (accumulate) {
                const uint32_t old = *q;
                g0 += __uint_as_float(old << 16);
                g1 += __uint_as_float(old & 0xFFFF0000u);
            }
            *q = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(g0)) |
                 ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(g1)) << 16);
        } else {
            if (ok0) {
                if (accumulate) g0 += __uint_as_float((uint32_t)p[0] << 16);
                p[0] = __bfloat16_as_ushort(__float2bfloat16_rn(g0));
            }
            if (ok1) {
                if (accumulate) g1 += __uint_as_float((uint32_t)p[1] << 16);
                p[1] = __bfloat16_as_ushort(__float2bfloat16_rn(g1));
            }
        }
    }
}

template <typename TG, bool GRAD, bool HIST>
__global__ void __launch_bounds__(kTailThreads, kCtasPerSm) chan_tail_kernel(const ChanArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TailSmem &sm = *reinterpret_cast<TailSmem *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t n_strips = (a.cols + kChanStrip - 1) / kChanStrip;
    const int64_t n_items = n_strips * a.n_slices;
    const uint32_t flip = a.lambda < 0.0 ? 0x80000000u : 0u;

    // count window: the symbols [-kSymWin/2, kSymWin/2) that the clamp leaves alone
    const int32_t wlo = (int32_t)max((int64_t)-kSymWin / 2, (int64_t)a.qmin);
    const int32_t whi = (int32_t)max((int64_t)wlo, min((int64_t)kSymWin / 2, (int64_t)a.qmax + 1));
    const float inv = (float)(1.0 / (double)a.step);
    // |t| below this is inside the window for sure; one compare per block of rows finds the rest
    const uint32_t near_bits = (wlo < 0 && whi > 0) ? __float_as_uint((float)min(-wlo, whi)) : 0u;
    unsigned long long *hist = reinterpret_cast<unsigned long long *>(a.hist);

    ChanLane ln;
    ln.a_addr[0] = (uint32_t)__cvta_generic_to_shared(&sm.a1[0][0][lane]);
    ln.a_addr[1] = (uint32_t)__cvta_generic_to_shared(&sm.a1[1][0][lane]);
    ln.b_addr[0] = (uint32_t)__cvta_generic_to_shared(&sm.bt[0][0][lane]);
    ln.b_addr[1] = (uint32_t)__cvta_generic_to_shared(&sm.bt[1][0][lane]);
    ln.e_lo = 1u;
    ln.inv = inv;
    ln.t_lo = (float)wlo - 0.5f;
    ln.t_hi = (float)whi;
    // floor(tc) lies in [wlo - 1, whi]; cell = floor(tc) - (wlo - 1)
    ln.cnt_off = (uint32_t)__cvta_generic_to_shared(sm.cnt) - (kMagicBits + (uint32_t)(wlo - 1)) * 4u;

    if constexpr (HIST) {
        for (int i = tid; i < kSymWin + 2; i += kTailThreads) sm.cnt[i] = 0u;
        if (tid < 2) sm.clampc[tid] = 0u;
    }
    if (tid < 128) sm.lg[tid] = log2(1.0 + (double)tid * (1.0 / 128.0));
    const bool vec_in = ((reinterpret_cast<uintptr_t>(a.x) & 3u) == 0) && ((a.ld & 1) == 0) && ((a.cols & 1) == 0);
    const bool vec_out = ((reinterpret_cast<uintptr_t>(a.grad) & (2 * sizeof(TG) - 1)) == 0) && ((a.grad_ld & 1) == 0) &&
                         ((a.cols & 1) == 0);
    const bool accumulate = a.accumulate != 0;
    int64_t cur_strip = -1;

    for (int64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
        // neighbouring CTAs take neighbouring strips of the same rows: their row pieces are adjacent in memory
        const int64_t strip = item % n_strips, slice = item / n_strips;
        const int64_t r_begin = a.rows * slice / a.n_slices, r_end = a.rows * (slice + 1) / a.n_slices;
        const int64_t c0 = strip * kChanStrip + 2 * lane;
        const bool ok0 = c0 < a.cols, ok1 = c0 + 1 < a.cols;

        if (GRAD && strip != cur_strip) {
            // ---- the tables of this strip's 64 columns
            cur_strip = strip;
            __syncthreads();
            if (tid == 0) sm.e_top = 0;
            __syncthreads();
            if (tid < kChanStrip) {
                const int64_t c = strip * kChanStrip + tid;
                const bool ok = c < a.cols;
                sm.colL[tid] = ok ? a.L[c] : __longlong_as_double(0x7FF8000000000000ll);
                sm.colb[tid] = ok ? a.b[c] : 0.0;
                if (ok) atomicMax(&sm.e_top, (int)(__float_as_uint(a.amax[c]) >> 23));
            }
            __syncthreads();
            const int e_lo = max(1, min(sm.e_top, 254) - (kAWin - 1));
            ln.e_lo = (uint32_t)e_lo;
            for (int idx = tid; idx < 2 * (kAWin + 1) * 32; idx += kTailThreads) {
                const int l = idx & 31, i = (idx >> 5) % (kAWin + 1), k = idx / (32 * (kAWin + 1));
                const double L = sm.colL[2 * l + k], b = sm.colb[2 * l + k];
                float v = 0.0f;                                  // a column without gradient: zero everywhere
                if (L == L) {
                    // One fp32 factor serves an exponent if the product with B stays in the normal range
                    // (|L + b (e-127)| <= 100); the rest, and the last row, hold the marker.
                    const int e = e_lo + i;
                    const double e0 = L + b * (double)(e - 127);
                    v = __int_as_float(0x7FC00000);
                    if (i < kAWin && e <= 254 && fabs(e0) <= 100.0)
                        v = __uint_as_float(__float_as_uint((float)exp2_short(e0)) ^ flip);
                }
                sm.a1[k][i][l] = v;
            }
            for (int idx = tid; idx < 2 * 128 * 32; idx += kTailThreads) {
                const int l = idx & 31, j = (idx >> 5) & 127, k = idx >> 12;
                const double L = sm.colL[2 * l + k], b = sm.colb[2 * l + k];
                sm.bt[k][j][l] = (L == L) ? (float)exp2_short(b * sm.lg[j]) : 1.0f;
            }
            __syncthreads();
        }

        // ---- stream the rows of the slice: warp w takes rows r_begin + w, + kTailWarps, ...
        const uint16_t *col = a.x + c0;
        TG *gcol = GRAD && a.grad != nullptr ? reinterpret_cast<TG *>(a.grad) + c0 : nullptr;
        double pen[2] = {0.0, 0.0};
        for (int64_t r = r_begin + warp; r < r_end; r += (int64_t)kTailWarps * kU) {
            const int nvalid = (int)min((int64_t)kU, (r_end - r + kTailWarps - 1) / kTailWarps);
            uint32_t w[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u)
                w[u] = u < nvalid ? load_pair(col + (r + (int64_t)u * kTailWarps) * a.ld, vec_in, ok0, ok1) : 0u;
            float g[kU][2];
            float mp[2] = {0.0f, 0.0f};
            uint32_t anyc = 0u;
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                g[u][0] = chan_elem<GRAD, HIST, 0>(w[u], ok0 && u < nvalid, ln, mp[0], anyc);
                g[u][1] = chan_elem<GRAD, HIST, 1>(w[u], ok1 && u < nvalid, ln, mp[1], anyc);
            }
            if constexpr (GRAD) {
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    if (mp[k] <= FLT_MAX) {
                        pen[k] += (double)mp[k];
                    } else {
                        // a marker, or a product beyond the fp32 range: this column's rows again, exactly
                        const double L = sm.colL[2 * lane + k], b = sm.colb[2 * lane + k];
                        pen[k] += chan_pen_exact(w, k, L, b);
#pragma unroll
                        for (int u = 0; u < kU; ++u) {
                            const uint32_t h = k ? (w[u] >> 16) : (w[u] & 0xFFFFu);
                            const uint32_t mag = h & 0x7FFFu;
                            const uint32_t i = min((mag >> 7) - ln.e_lo, (uint32_t)kAWin);
                            const float av = lds_f32(ln.a_addr[k] + i * 128u);
                            if (av != av && mag != 0u)
                                g[u][k] = __uint_as_float(__float_as_uint(chan_grad_exact(mag, L, b, flip)) ^ ((h & 0x8000u) << 16));
                        }
                    }
                }
            }
            if constexpr (HIST) {
                if (anyc >= near_bits) {
                    // some element may have missed the window (its count went to a sentinel): exact test, slow count
                    for (int u = 0; u < nvalid; ++u) {
                        for (int k = 0; k < 2; ++k) {
                            if (!(k ? ok1 : ok0)) continue;
                            const float x = __uint_as_float(k ? (w[u] & 0xFFFF0000u) : (w[u] << 16));
                            const float t = __fmul_rn(x, inv);
                            if (!(t >= (float)wlo && t < (float)whi))
                                chan_count_slow(x, inv, a.qmin, a.qmax, wlo, whi, sm, hist);
                        }
                    }
                }
            }
            if constexpr (GRAD) {
                if (gcol != nullptr) {
#pragma unroll
                    for (int u = 0; u < kU; ++u)
                        if (u < nvalid)
                            store_pair<TG>(gcol + (r + (int64_t)u * kTailWarps) * a.grad_ld, g[u][0], g[u][1], vec_out, ok0, ok1,
                                           accumulate);
                }
            }
        }

        if constexpr (GRAD) {
            // penalty partial of every column of the strip: the warps in a fixed order
            sm.red[warp][2 * lane] = pen[0];
            sm.red[warp][2 * lane + 1] = pen[1];
            __syncthreads();
            if (tid < kChanStrip) {
                const int64_t c = strip * kChanStrip + tid;
                if (c < a.cols) {
                    double p = 0.0;
                    for (int wv = 0; wv < kTailWarps; ++wv) p += sm.red[wv][tid];
                    a.pen[slice * a.cols + c] = p;
                }
            }
            __syncthreads();
        }
    }

    if constexpr (HIST) {
        __syncthreads();
        const int n_cells = whi - wlo;
        for (int i = tid; i < n_cells; i += kTailThreads) {
            // (every CTA starts at another cell: CTAs that finish together do not walk the bins in step)
            const int cidx = (int)(((uint32_t)i + blockIdx.x * 61u) % (uint32_t)n_cells);
            const uint32_t n = sm.cnt[cidx + 1];
            if (n != 0u) atomicAdd(&hist[(wlo + cidx) - a.qmin], (unsigned long long)n);
        }
        if (tid < 2 && a.clamped != nullptr && sm.clampc[tid] != 0u)
            atomicAdd(reinterpret_cast<unsigned long long *>(a.clamped) + tid, (unsigned long long)sm.clampc[tid]);
    }
}

template <typename TG>
cudaError_t launch_tail_typed(const ChanArgs &a, int grid, cudaStream_t st)
{
    void (*kern)(const ChanArgs) = nullptr;
    if (a.do_grad && a.do_hist) kern = chan_tail_kernel<TG, true, true>;
    else if (a.do_grad) kern = chan_tail_kernel<TG, true, false>;
    else kern = chan_tail_kernel<TG, false, true>;
    // more than 48 KB of dynamic shared memory needs the opt-in (per function and device)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TailSmem));
    if (e != cudaSuccess) return e;
    kern<<<grid, kTailThreads, sizeof(TailSmem), st>>>(a);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_chan_moments(const ChanArgs &a, cudaStream_t st)
{
    if (a.rows <= 0 || a.cols <= 0) return cudaSuccess;
    const dim3 grid((unsigned)((a.cols + kChanStrip - 1) / kChanStrip), (unsigned)a.n_mom_blocks);
    chan_moments_kernel<<<grid, kMomThreads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_chan_fit(const ChanArgs &a, cudaStream_t st)
{
    if (a.cols <= 0) return cudaSuccess;
    chan_fit_kernel<<<(unsigned)((a.cols + 127) / 128), 128, 0, st>>>(a);
    return cudaGetLastError();
}

// Row slices per strip: enough items to fill two CTAs per SM, in whole rounds of the grid where
// there are more items than CTAs, and at least 512 rows per item so that the tables (192 entries
// per column) stay cheap next to the rows they serve.
int chan_slices(int64_t rows, int64_t cols, int sm_count)
{
    const int64_t n_strips = (cols + kChanStrip - 1) / kChanStrip;
    const int64_t slots = (int64_t)sm_count * kCtasPerSm;
    const int64_t most = rows / 512 > 1 ? rows / 512 : 1;
    int64_t best = 1;
    double best_fill = 0.0;
    for (int64_t ns = 1; ns <= most && ns <= 64; ++ns) {
        const int64_t items = n_strips * ns;
        const int64_t rounds = (items + slots - 1) / slots;
        const double fill = (double)items / (double)(rounds * slots);
        if (fill > best_fill + 0.02) { best_fill = fill; best = ns; }
    }
    return (int)best;
}

cudaError_t launch_chan_tail(gg_dtype grad_dtype, const ChanArgs &a, int sm_count, cudaStream_t st)
{
    if (a.rows <= 0 || a.cols <= 0 || (!a.do_grad && !a.do_hist)) return cudaSuccess;
    const int64_t n_items = (a.cols + kChanStrip - 1) / kChanStrip * a.n_slices;
    const int grid = (int)min(n_items, (int64_t)sm_count * kCtasPerSm);
    if (a.grad != nullptr && grad_dtype == GG_BF16) return launch_tail_typed<uint16_t>(a, grid, st);
    return launch_tail_typed<float>(a, grid, st);
}

cudaError_t launch_chan_penalty(const ChanArgs &a, cudaStream_t st)
{
    if (a.cols <= 0 || a.penalty == nullptr) return cudaSuccess;
    chan_penalty_kernel<<<(unsigned)((a.cols + 127) / 128), 128, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace gg
