// The GG pass over the COLUMNS of a row-major bf16 matrix (one generalized Gaussian per channel).
//
// A column is a strided segment, so the kernels are tiled the other way round from the contiguous
// path: a strip of 64 neighbouring columns is 128 contiguous bytes of every row, a warp reads one
// such row piece per load (lane l holds columns 2l and 2l+1 as one 32-bit word) and walks down the
// rows, so every thread accumulates the sums of its own two columns and no transposition happens.
//   chan_moments_kernel   one CTA per (strip, block of 512 rows): sum |x|, sum x^2, non-finite
//                         count, min, max per column, written per row block
//   chan_fit_kernel       16 threads per column: add the row blocks in a fixed order, invert the moment
//                         ratio from the fit table, derive the constants of the gradient
//   chan_tables_kernel    one CTA per strip: the per-column gradient tables |g| = A_c[e] * B_c[j]
//                         (e exponent field, j mantissa bits of the bf16 pattern), laid out so that
//                         lane l reads word l of a table row: no look-up ever meets a bank conflict
//   chan_tail_kernel      persistent CTAs over (strip, slice of rows) items: copy the strip's tables
//                         to shared memory, then stream the rows: gradient, penalty partial per
//                         column, counts in shared memory
//   chan_penalty_kernel   one thread per column: adds the slices in order, divides by beta
// Both sweeps read through per-thread rings of asynchronous 4-byte copies (two blocks of eight rows),
// so the rows in flight cost no registers.
// A is kept for a window of 64 exponents below the largest magnitude of the strip; every exponent
// outside it, zero/subnormal/inf/nan and far binades read a NaN marker, the NaN reaches the
// column's penalty partial of the current block of rows, and the range check of that partial
// sends the block's column to an exact fp64 path.  Exact zeros are common in activations and are
// selected to a zero gradient without the exact path.
// Counts: by symbol in a 4096-cell window while that reaches 6.5 standard deviations of the strip's
// widest column, else by bf16 bit pattern over the binades up to the strip's largest magnitude,
// quantised when the cells are flushed.  An element outside the window in use counts in a sentinel
// cell and is counted again, one by one, after its block of rows.
#include <cuda_bf16.h>
#include <float.h>

#include <type_traits>

#include "gg_fit_table.cuh"
#include "gg_device.cuh"
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
constexpr int kSlowWin = 512;                  // symbols [-256, 256) of the one-by-one path in pattern counting
// Pattern counting: one cell per bf16 magnitude pattern and sign over 16 binades, one cell for zero.
constexpr uint32_t kPatCells = 16 * 128;       // magnitude patterns in the window: cell pairs 0 .. kPatCells - 1
constexpr uint32_t kPatZero = kPatCells;       // the cell pair of +-0
constexpr uint32_t kPatSentinel = kPatCells + 1;
static_assert((kPatSentinel + 1) * 2 <= kSymWin + 4, "the pattern cells share the symbol cells' array");

// The 32-bit word of columns (2 lane, 2 lane + 1) of one row; missing columns read as zero.
__device__ __forceinline__ uint32_t load_pair(const uint16_t *row, bool vec, bool ok0, bool ok1)
{
    if (vec) return ok0 ? __ldg(reinterpret_cast<const uint32_t *>(row)) : 0u;   // (vec: cols is even, ok0 == ok1)
    uint32_t w = 0;
    if (ok0) w = (uint32_t)__ldg(row);
    if (ok1) w |= (uint32_t)__ldg(row + 1) << 16;
    return w;
}

// One element in fp64; a non-finite entry is counted and left out (used when the fp32 partials of a
// block of rows cannot stand for the exact sums).
__device__ __forceinline__ void moments_careful(uint32_t h, double &s1, double &s2, uint32_t &bad)
{
    const uint32_t mag = h & 0x7FFFu;
    if (mag < 0x7F80u) {
        const double ax = (double)__uint_as_float(mag << 16);
        s1 += ax;
        s2 += ax * ax;
    } else {
        bad += 1u;
    }
}

// kU rows of the lane's two columns (row u is the 32-bit word word_of(u); rows past the end and missing
// columns read as zero, which adds nothing to the sums; the caller repairs the extremes) into the
// running sums.
template <typename WordOf>
__device__ __forceinline__ void mom_block(WordOf word_of, double (&s1)[2], double (&s2)[2], uint32_t (&bad)[2],
                                          __nv_bfloat162 &mn2, __nv_bfloat162 &mx2)
{
    float m1[2] = {0.0f, 0.0f}, m2[2] = {0.0f, 0.0f};
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const uint32_t w = word_of(u);
        const float lo = __uint_as_float(w << 16), hi = __uint_as_float(w & 0xFFFF0000u);
        m1[0] += fabsf(lo);
        m2[0] = fmaf(lo, lo, m2[0]);
        m1[1] += fabsf(hi);
        m2[1] = fmaf(hi, hi, m2[1]);
        const __nv_bfloat162 pr = *reinterpret_cast<const __nv_bfloat162 *>(&w);
        mn2 = __hmin2(mn2, pr);
        mx2 = __hmax2(mx2, pr);
    }
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        if (run_sums_exact_enough(m1[k], m2[k])) {
            s1[k] += (double)m1[k];
            s2[k] += (double)m2[k];
        } else {     // an inf or nan (left out of the sums and counted), or squares outside the fp32 range
#pragma unroll
            for (int u = 0; u < kU; ++u) moments_careful(k ? (word_of(u) >> 16) : word_of(u), s1[k], s2[k], bad[k]);
        }
    }
}

__global__ void __launch_bounds__(kMomThreads, 5) chan_moments_kernel(const ChanArgs a)
{
    __shared__ double red1[kMomWarps][kChanStrip], red2[kMomWarps][kChanStrip];
    __shared__ uint32_t redb[kMomWarps][kChanStrip];
    __shared__ float redmn[kMomWarps][kChanStrip], redmx[kMomWarps][kChanStrip];
    __shared__ uint32_t ring[2][kU][kMomThreads];     // per-thread slots of the rows in flight
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kChanStrip + 2 * lane;
    const int64_t r_begin = (int64_t)blockIdx.y * kChanMomRows;
    const int64_t r_end = min(a.rows, r_begin + kChanMomRows);
    const bool ok0 = c0 < a.cols, ok1 = c0 + 1 < a.cols;
    const bool vec = ((reinterpret_cast<uintptr_t>(a.x) & 3u) == 0) && ((a.ld & 1) == 0) && ((a.cols & 1) == 0);
    const uint16_t *col = a.x + c0;

    double s1[2] = {0.0, 0.0}, s2[2] = {0.0, 0.0};
    uint32_t bad[2] = {0u, 0u};
    // extremes of both columns at once, as packed bf16 (min and max return the non-NaN operand, like fminf)
    __nv_bfloat162 mn2 = __floats2bfloat162_rn(INFINITY, INFINITY), mx2 = __floats2bfloat162_rn(-INFINITY, -INFINITY);
    const int64_t stride = (int64_t)kMomWarps * a.ld;
    const int64_t r0 = r_begin + warp;
    const uint16_t *p = col + r0 * a.ld;
    int n_mine = r0 < r_end ? (int)((r_end - r0 + kMomWarps - 1) / kMomWarps) : 0;      // rows of this warp
    if (vec && ok0) {
        // Whole blocks of kU rows: the thread stages its words of the next block in its own ring slots with
        // asynchronous copies while it sums the current one (one commit group per block, so the group that
        // must have landed is always the one before the last).
        const uint32_t slot = (uint32_t)__cvta_generic_to_shared(&ring[0][0][threadIdx.x]);
        constexpr uint32_t kRow = kMomThreads * 4u;
        const int n_blocks = n_mine / kU;
        auto stage = [&](const uint16_t *src, uint32_t dst) {
#pragma unroll
            for (int u = 0; u < kU; ++u)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst + (uint32_t)u * kRow), "l"(src + u * stride) : "memory");
        };
        if (n_blocks > 0) stage(p, slot);
        asm volatile("cp.async.commit_group;" ::: "memory");
        for (int bk = 0; bk < n_blocks; ++bk) {
            const uint32_t cur = slot + (uint32_t)(bk & 1) * kU * kRow;
            if (bk + 1 < n_blocks) stage(p + kU * stride, slot + (uint32_t)((bk + 1) & 1) * kU * kRow);
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 1;" ::: "memory");
            mom_block([&](int u) {
                uint32_t w;
                asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(cur + (uint32_t)u * kRow));
                return w;
            }, s1, s2, bad, mn2, mx2);
            p += kU * stride;
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        n_mine -= n_blocks * kU;
    }
    for (; n_mine > 0; n_mine -= kU, p += kU * stride) {
        uint32_t w[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) w[u] = u < n_mine ? load_pair(p + u * stride, vec, ok0, ok1) : 0u;
        mom_block([&](int u) { return w[u]; }, s1, s2, bad, mn2, mx2);
    }
    float mn[2] = {__low2float(mn2), __high2float(mn2)}, mx[2] = {__low2float(mx2), __high2float(mx2)};
    // Rows past the end and missing columns entered the extremes as zeros.  Only the last row block and
    // the last strip can have them: there the extremes are taken again over the real entries alone.
    if (r_end - r_begin < kChanMomRows || !ok0 || !ok1) {
        mn[0] = mn[1] = INFINITY;
        mx[0] = mx[1] = -INFINITY;
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

// 32 columns per CTA, 16 threads per column: thread (column, g) adds the row blocks g, g + 16, ... in
// order, thread (column, 0) adds the 16 partial sums in order and does the fit, the clamp flag and the
// gradient constants.
constexpr int kFitCols = 32, kFitGroups = 16;
__global__ void __launch_bounds__(kFitCols * kFitGroups) chan_fit_kernel(const ChanArgs a)
{
    __shared__ double r1[kFitGroups][kFitCols], r2[kFitGroups][kFitCols];
    __shared__ uint32_t rb[kFitGroups][kFitCols];
    __shared__ float rmn[kFitGroups][kFitCols], rmx[kFitGroups][kFitCols];
    __shared__ int need[kFitCols];
    const int cx = threadIdx.x % kFitCols, grp = threadIdx.x / kFitCols;
    const int64_t c = (int64_t)blockIdx.x * kFitCols + cx;
    double s1 = 0.0, s2 = 0.0;
    uint32_t bad = 0;
    float xmin = INFINITY, xmax = -INFINITY;
    if (c < a.cols) {
#pragma unroll 4
        for (int k = grp; k < a.n_mom_blocks; k += kFitGroups) {
            const int64_t o = (int64_t)k * a.cols + c;
            s1 += a.s1[o]; s2 += a.s2[o]; bad += a.bad[o];
            xmin = fminf(xmin, a.xmin[o]); xmax = fmaxf(xmax, a.xmax[o]);
        }
    }
    r1[grp][cx] = s1; r2[grp][cx] = s2; rb[grp][cx] = bad; rmn[grp][cx] = xmin; rmx[grp][cx] = xmax;
    __syncthreads();
    const bool lead = grp == 0 && c < a.cols;
    if (grp == 0) need[cx] = 0;
    if (lead) {
        for (int g = 1; g < kFitGroups; ++g) {
            s1 += r1[g][cx]; s2 += r2[g][cx]; bad += rb[g][cx];
            xmin = fminf(xmin, rmn[g][cx]); xmax = fmaxf(xmax, rmx[g][cx]);
        }
        // an ill-conditioned fit of a short column (see careful_sums): its sums again in fp64, by the column's 16 threads
        if (a.rows > 0 && a.rows <= kCarefulLen && s2 > 0.0) {
            const double m1 = s1 / (double)a.rows, m2 = s2 / (double)a.rows;
            need[cx] = log(m1 * m1 / m2) > kCarefulLogRatio;
        }
    }
    __syncthreads();
    if (c < a.cols && need[cx]) {
        double t1 = 0.0, t2 = 0.0;
        for (int64_t r = grp; r < a.rows; r += kFitGroups) {
            double ax;
            bool fin;
            if (a.in_f32) {
                const uint32_t ab = __float_as_uint(__ldg(reinterpret_cast<const float *>(a.x) + r * a.ld + c)) & 0x7FFFFFFFu;
                fin = ab < 0x7F800000u;
                ax = (double)__uint_as_float(ab);
            } else {
                const uint32_t h = (uint32_t)__ldg(a.x + r * a.ld + c) & 0x7FFFu;
                fin = h < 0x7F80u;
                ax = (double)__uint_as_float(h << 16);
            }
            if (fin) { t1 += ax; t2 = fma(ax, ax, t2); }
        }
        r1[grp][cx] = t1;
        r2[grp][cx] = t2;
    }
    __syncthreads();
    if (!lead) return;
    if (need[cx]) {
        s1 = r1[0][cx]; s2 = r2[0][cx];
        for (int g = 1; g < kFitGroups; ++g) { s1 += r1[g][cx]; s2 += r2[g][cx]; }
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
    // the standard deviation decides how the second kernel counts this column's strip
    const double sd = a.rows > 0 ? sqrt(s2 / (double)a.rows) : 0.0;
    a.sd[c] = sd <= (double)FLT_MAX ? (float)sd : FLT_MAX;
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

// Warp-uniform constants that only the cold paths need.
struct ChanConst {
    float inv;
    int32_t wlo, whi, qmin, qmax;     // count window [wlo, whi), clamp
    uint32_t flip;                    // sign bit of lambda
    unsigned long long *hist;
};

constexpr int kTabFloats = 2 * (kAWin + 1) * 32 + 2 * 128 * 32;     // one strip's A and B tables
static_assert(kTabFloats == kChanTabFloats && kTabFloats % 4 == 0, "table layout");

struct TailSmem {
    uint32_t ring[2][kU][kTailThreads];   // per-thread slots of the rows in flight: two blocks of kU rows
    float a1[2][kAWin + 1][32];       // [k][e - e_lo][lane]: A of column 2 lane + k; row kAWin: the marker
    float bt[2][128][32];             // [k][j][lane]: B of column 2 lane + k
    uint32_t cnt[kSymWin + 4];        // symbol counting: cell 0 and cell whi - wlo + 1 are the sentinels of the two tails;
                                      // pattern counting: word (p * 2 + sign), p < kPatCells: the window's patterns, p = kPatZero: zero, p = kPatSentinel: the sentinel
    double red[kTailWarps][kChanStrip];
    double colL[kChanStrip], colb[kChanStrip];
    uint32_t win[kSlowWin];           // pattern counting: symbols [-kSlowWin/2, kSlowWin/2) of the slow path
    uint32_t clampc[2];
    int amax_bits, sd_bits;           // largest finite magnitude and largest standard deviation of the current strip's columns (bits of floats)
    ChanConst cc;
};

// Exact gradient magnitude (with lambda's sign through `flip`) of a 15-bit magnitude pattern.
__device__ __noinline__ float chan_grad_exact(uint32_t mag, double L, double b, uint32_t flip)
{
    const float ax = __uint_as_float(mag << 16);
    if (!(L == L) || ax == 0.0f) return 0.0f;
    const float v = (float)exp2(L + b * log2((double)ax));
    return __uint_as_float(__float_as_uint(v) ^ flip);
}

// fp64 penalty term |x| |g| of one magnitude pattern.
__device__ __noinline__ double chan_pen_exact(uint32_t mag, double L, double b)
{
    const double ax = (double)__uint_as_float(mag << 16);
    if (!(L == L) || ax == 0.0) return 0.0;
    return ax * exp2(L + b * log2(ax));
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
        // wlo < whi: symbol counting, whose cells the slow path may use; else the small window of its own
        if (q >= wlo && q < whi) atomicAdd(&sm.cnt[q - wlo + 1], 1u);
        else if (wlo >= whi && (uint32_t)(q + kSlowWin / 2) < (uint32_t)kSlowWin) atomicAdd(&sm.win[q + kSlowWin / 2], 1u);
        else atomicAdd(&hist[q - qmin], 1ull);
    }
}

// One CTA per strip: the gradient tables of its 64 columns, in the layout of TailSmem::a1 and bt,
// and the exponent field of the first A row.
__global__ void __launch_bounds__(kTailThreads) chan_tables_kernel(const ChanArgs a)
{
    __shared__ double colL[kChanStrip], colb[kChanStrip], lg[128];
    __shared__ int e_top;
    const int tid = threadIdx.x, strip = blockIdx.x;
    const uint32_t flip = a.lambda < 0.0 ? 0x80000000u : 0u;
    if (tid == 0) e_top = 0;
    if (tid < 128) lg[tid] = log2(1.0 + (double)tid * (1.0 / 128.0));
    __syncthreads();
    if (tid < kChanStrip) {
        const int64_t c = (int64_t)strip * kChanStrip + tid;
        const bool ok = c < a.cols;
        colL[tid] = ok ? a.L[c] : __longlong_as_double(0x7FF8000000000000ll);
        colb[tid] = ok ? a.b[c] : 0.0;
        if (ok) atomicMax(&e_top, (int)(__float_as_uint(a.amax[c]) >> 23));
    }
    __syncthreads();
    // the window: 64 exponents up to that of the largest magnitude of the strip
    const int e_lo = max(1, min(e_top, 254) - (kAWin - 1));
    if (tid == 0) a.tab_elo[strip] = e_lo;
    float *ta = a.tab + (int64_t)strip * kTabFloats, *tb = ta + 2 * (kAWin + 1) * 32;
    for (int idx = tid; idx < 2 * (kAWin + 1) * 32; idx += kTailThreads) {
        const int l = idx & 31, i = (idx >> 5) % (kAWin + 1), k = idx / (32 * (kAWin + 1));
        const double L = colL[2 * l + k], b = colb[2 * l + k];
        float v = 0.0f;                                  // a column without gradient: zero everywhere
        if (L == L) {
            // One fp32 factor serves an exponent if the product with B stays in the normal range
            // (|L + b (e-127)| <= 100); the rest, and the last row, hold the marker.
            const int e = e_lo + i;
            const double e0 = L + b * (double)(e - 127);
            v = __int_as_float(0x7FC00000);
            if (i < kAWin && e <= 254 && fabs(e0) <= 100.0) v = __uint_as_float(__float_as_uint((float)exp2_short(e0)) ^ flip);
        }
        ta[idx] = v;                                     // [k][i][l]
    }
    for (int idx = tid; idx < 2 * 128 * 32; idx += kTailThreads) {
        const int l = idx & 31, j = (idx >> 5) & 127, k = idx >> 12;
        const double L = colL[2 * l + k], b = colb[2 * l + k];
        tb[idx] = (L == L) ? (float)exp2_short(b * lg[j]) : 1.0f;      // [k][j][l]
    }
}

// Per-thread constants of the element path (the rest lives in TailSmem::cc).
struct ChanLane {
    uint32_t a_addr, b_addr;         // shared-memory addresses of this lane's word in row 0 of its first tables
    uint32_t e_lo;                   // exponent field of row 0 of the A tables
    uint32_t cnt_off;                // symbol counting: cell of a value = bits(floor(t) + magic) * 4 + cnt_off (mod 2^32)
    uint32_t cnt_addr, cbase;        // pattern counting: address of cnt, first magnitude pattern of the window
    float inv, t_lo, t_hi;           // quantiser scale; t is clamped to [t_lo, t_hi] so that its floor is a cell
    float near;                      // a smaller |t| lies inside the count window for sure
};
constexpr uint32_t kA2 = (kAWin + 1) * 128u;     // byte offset of the second column's A table
constexpr uint32_t kB2 = 128u * 128u;            // and of its B table

// Row i of the lane's A table / row j of its B table for column HALF.
template <int HALF>
__device__ __forceinline__ float lds_a(const ChanLane &ln, uint32_t i)
{
    float v;
    asm("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(ln.a_addr + i * 128u), "n"(HALF ? kA2 : 0u));
    return v;
}
template <int HALF>
__device__ __forceinline__ float lds_b(const ChanLane &ln, uint32_t j)
{
    float v;
    asm("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(ln.b_addr + j * 128u), "n"(HALF ? kB2 : 0u));
    return v;
}

// One element (HALF 0: the low half of w, the lane's even column).  Branch free.
template <bool GRAD, bool HIST, bool PAT, int HALF>
__device__ __forceinline__ float chan_elem(uint32_t w, bool counted, const ChanLane &ln, float &mp, float &anyc)
{
    const uint32_t xb = HALF ? (w & 0xFFFF0000u) : (w << 16);
    float g = 0.0f;
    if constexpr (GRAD) {
        const uint32_t e = HALF ? (w >> 23) & 0xFFu : (w >> 7) & 0xFFu;
        const uint32_t j = HALF ? (w >> 16) & 127u : w & 127u;
        const uint32_t i = min(e - ln.e_lo, (uint32_t)kAWin);       // below the window wraps around to the marker too
        float ga = lds_a<HALF>(ln, i) * lds_b<HALF>(ln, j);
        ga = (xb << 1) == 0u ? 0.0f : ga;                            // g(0) = 0 for every shape
        mp = fmaf(fabsf(__uint_as_float(xb)), fabsf(ga), mp);
        g = __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));   // the table carries lambda's sign
    }
    if constexpr (HIST) {
        if (counted && PAT) {
            // by bit pattern: anyc keeps the largest window index (as the bits of a float, whose order they share)
            const uint32_t mag = HALF ? (w >> 16) & 0x7FFFu : w & 0x7FFFu;
            // (below the window the difference wraps around to the sentinel too; the window is placed so that no
            // element has the pattern cbase + kPatCells, which would fall on the zero cell)
            uint32_t pc = min(mag - ln.cbase, kPatSentinel);
            pc = mag == 0u ? kPatZero : pc;
            anyc = __uint_as_float(max(__float_as_uint(anyc), pc));
            const uint32_t sign4 = HALF ? (w >> 29) & 4u : (w >> 13) & 4u;
            red_inc(ln.cnt_addr + pc * 8u + sign4);
        } else if (counted) {
            const float t = __fmul_rn(__uint_as_float(xb), ln.inv);
            anyc = fmaxf(anyc, fabsf(t));      // (a nan is ignored here and lands on a sentinel: nan is not counted)
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
__device__ __forceinline__ void store_one(TG *p, float g)
{
    if constexpr (sizeof(TG) == 4) *p = g;
    else *p = __bfloat16_as_ushort(__float2bfloat16_rn(g));
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

// The exact path of one column (HALF) of a block of rows whose fp32 penalty partial is not a usable
// number (a marker, or a product beyond the fp32 range): fp64 penalty terms of all its rows, and the
// exact gradient of every element that read a marker, handed to `fix(u, g)`.
template <int HALF, typename WordOf, typename Fix>
__device__ __forceinline__ double chan_column_exact(const ChanLane &ln, const TailSmem &sm, int lane, WordOf word_of, Fix fix)
{
    const double L = sm.colL[2 * lane + HALF], b = sm.colb[2 * lane + HALF];
    double dp = 0.0;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const uint32_t w = word_of(u);
        const uint32_t h = HALF ? (w >> 16) : (w & 0xFFFFu);
        const uint32_t mag = h & 0x7FFFu;
        dp += chan_pen_exact(mag, L, b);                       // (rows past the end read as zero: no term)
        const float av = lds_a<HALF>(ln, min((mag >> 7) - ln.e_lo, (uint32_t)kAWin));
        if (av != av && mag != 0u)
            fix(u, __uint_as_float(__float_as_uint(chan_grad_exact(mag, L, b, sm.cc.flip)) ^ ((h & 0x8000u) << 16)));
    }
    return dp;
}

// Elements of a block whose count may have gone to a sentinel: exact test, slow count.
template <bool PAT, typename WordOf, typename Counted>
__device__ __forceinline__ void chan_recount(TailSmem &sm, uint32_t cbase, WordOf word_of, Counted counted)
{
    const float inv = sm.cc.inv;
    const int32_t wlo = sm.cc.wlo, whi = sm.cc.whi;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const uint32_t w = word_of(u);
            const float x = __uint_as_float(k ? (w & 0xFFFF0000u) : (w << 16));
            const float t = __fmul_rn(x, inv);
            bool miss;
            if constexpr (PAT) {
                const uint32_t mag = (k ? (w >> 16) : w) & 0x7FFFu;
                miss = mag != 0u && mag - cbase >= kPatCells;
            } else {
                miss = !(t >= (float)wlo && t < (float)whi);
            }
            if (counted(u, k) && miss) {
                if constexpr (PAT) {
                    // most misses are small values below the pattern window: their few symbols meet in the small
                    // window, without a call
                    const int q = __float2int_rd(t);
                    if (t == t && (uint32_t)(q + kSlowWin / 2) < (uint32_t)kSlowWin && q >= sm.cc.qmin && q <= sm.cc.qmax) {
                        atomicAdd(&sm.win[q + kSlowWin / 2], 1u);
                        continue;
                    }
                }
                // (the slow count may only use the shared cells in symbol counting: wlo = whi switches that off)
                chan_count_slow(x, inv, sm.cc.qmin, sm.cc.qmax, PAT ? 0 : wlo, PAT ? 0 : whi, sm, sm.cc.hist);
            }
        }
    }
}

// kU whole rows of a whole strip, staged in this thread's ring slots at shared address wbase (row u
// at wbase + u * kRowBytes).  The gradient pair of a row is written as soon as it is known; an element
// the tables could not serve is written again, alone, by the exact path.
constexpr uint32_t kRowBytes = kTailThreads * 4u;
template <typename TG, bool GRAD, bool HIST, bool PAT>
__device__ __forceinline__ void chan_block_fast(uint32_t wbase, TG *gp, int64_t sg, int lane, const ChanLane &ln, TailSmem &sm,
                                                double (&pen)[2])
{
    auto word_of = [&](int u) {
        uint32_t w;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(wbase + (uint32_t)u * kRowBytes));
        return w;
    };
    float mp[2] = {0.0f, 0.0f};
    float anyc = 0.0f;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const uint32_t w = word_of(u);
        const float g0 = chan_elem<GRAD, HIST, PAT, 0>(w, true, ln, mp[0], anyc);
        const float g1 = chan_elem<GRAD, HIST, PAT, 1>(w, true, ln, mp[1], anyc);
        if constexpr (GRAD) {
            if (gp != nullptr) store_pair<TG>(gp + u * sg, g0, g1, true, true, true, false);
        }
    }
    if constexpr (GRAD) {
        if (mp[0] <= FLT_MAX) pen[0] += (double)mp[0];
        else pen[0] += chan_column_exact<0>(ln, sm, lane, word_of, [&](int u, float g) { if (gp != nullptr) store_one<TG>(gp + u * sg, g); });
        if (mp[1] <= FLT_MAX) pen[1] += (double)mp[1];
        else pen[1] += chan_column_exact<1>(ln, sm, lane, word_of, [&](int u, float g) { if (gp != nullptr) store_one<TG>(gp + u * sg + 1, g); });
    }
    if constexpr (HIST) {
        if (PAT ? __float_as_uint(anyc) >= kPatSentinel : anyc >= ln.near) chan_recount<PAT>(sm, ln.cbase, word_of, [](int, int) { return true; });
    }
}

// Adds the counted cells to the histogram and empties them (all threads; the caller has synchronised, so
// all counting under the current layout is complete).  Symbol cells hold symbols wlo .. whi - 1, which the
// clamp leaves alone; pattern cells are quantised here, one pattern at a time.
__device__ void chan_flush(TailSmem &sm, bool pat, uint32_t cbase, const ChanArgs &a)
{
    unsigned long long *hist = sm.cc.hist;
    if (pat) {
        for (uint32_t i = threadIdx.x; i < (kPatSentinel + 1) * 2; i += kTailThreads) {
            // (every CTA starts at another cell: CTAs that flush together do not walk the bins in step)
            const uint32_t cw = (i + blockIdx.x * 61u) % ((kPatSentinel + 1) * 2);
            const uint32_t n = sm.cnt[cw];
            if (n == 0u) continue;
            sm.cnt[cw] = 0u;
            const uint32_t pc = cw >> 1;
            if (pc == kPatSentinel) continue;          // counted again, one by one, by the slow path
            const uint32_t h = (pc == kPatZero ? 0u : cbase + pc) | ((cw & 1u) << 15);
            const float t = __fmul_rn(__uint_as_float(h << 16), sm.cc.inv);
            if (!(t == t)) continue;                   // (a window that reaches the top binade holds the nan patterns: not counted)
            int q = __float2int_rd(t);                 // floor, saturating
            if (q < sm.cc.qmin) { q = sm.cc.qmin; atomicAdd(&sm.clampc[0], n); }
            else if (q > sm.cc.qmax) { q = sm.cc.qmax; atomicAdd(&sm.clampc[1], n); }
            // many patterns below the step share the symbols around zero: those meet in the small window first
            if ((uint32_t)(q + kSlowWin / 2) < (uint32_t)kSlowWin) atomicAdd(&sm.win[q + kSlowWin / 2], n);
            else atomicAdd(&hist[q - sm.cc.qmin], (unsigned long long)n);
        }
        __syncthreads();
        for (int i = threadIdx.x; i < kSlowWin; i += kTailThreads) {      // (its symbols are already clamped)
            const uint32_t n = sm.win[i];
            if (n != 0u) {
                sm.win[i] = 0u;
                atomicAdd(&hist[(i - kSlowWin / 2) - sm.cc.qmin], (unsigned long long)n);
            }
        }
    } else {
        const int wlo = sm.cc.wlo, n_cells = sm.cc.whi - sm.cc.wlo;
        for (int i = threadIdx.x; i < n_cells + 2; i += kTailThreads) {
            const int cidx = (int)(((uint32_t)i + blockIdx.x * 61u) % (uint32_t)(n_cells + 2));
            const uint32_t n = sm.cnt[cidx];
            if (n == 0u) continue;
            sm.cnt[cidx] = 0u;
            if (cidx >= 1 && cidx <= n_cells) atomicAdd(&hist[(wlo + cidx - 1) - a.qmin], (unsigned long long)n);
        }
    }
    __syncthreads();
}

// Up to kU rows with every guard (ragged blocks, the last strip, unaligned rows, accumulation), as a
// call of its own so that its registers do not weigh on the streaming loop: rows past nvalid and
// missing columns read as zero and are not counted, and the gradients wait in registers until the
// exact path has run (they may have to be added to what is stored).  Returns the two penalty
// contributions.
template <typename TG, bool GRAD, bool HIST, bool PAT>
__device__ __noinline__ double2 chan_block_guarded(const uint16_t *p, int64_t sin, TG *gp, int64_t sg, int nvalid, bool ok0,
                                                   bool ok1, bool vec_in, bool vec_out, bool accumulate, int lane, ChanLane ln,
                                                   TailSmem *smp)
{
    TailSmem &sm = *smp;
    uint32_t w[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) w[u] = u < nvalid ? load_pair(p + u * sin, vec_in, ok0, ok1) : 0u;
    auto word_of = [&](int u) { return w[u]; };
    float g[kU][2];
    float mp[2] = {0.0f, 0.0f};
    float anyc = 0.0f;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        g[u][0] = chan_elem<GRAD, HIST, PAT, 0>(w[u], ok0 && u < nvalid, ln, mp[0], anyc);
        g[u][1] = chan_elem<GRAD, HIST, PAT, 1>(w[u], ok1 && u < nvalid, ln, mp[1], anyc);
    }
    double2 pen = make_double2(0.0, 0.0);
    if constexpr (GRAD) {
        if (mp[0] <= FLT_MAX) pen.x = (double)mp[0];
        else pen.x = chan_column_exact<0>(ln, sm, lane, word_of, [&](int u, float ge) { g[u][0] = ge; });
        if (mp[1] <= FLT_MAX) pen.y = (double)mp[1];
        else pen.y = chan_column_exact<1>(ln, sm, lane, word_of, [&](int u, float ge) { g[u][1] = ge; });
    }
    if constexpr (HIST) {
        if (PAT ? __float_as_uint(anyc) >= kPatSentinel : anyc >= ln.near)
            chan_recount<PAT>(sm, ln.cbase, word_of, [&](int u, int k) { return u < nvalid && (k ? ok1 : ok0); });
    }
    if constexpr (GRAD) {
        if (gp != nullptr) {
#pragma unroll
            for (int u = 0; u < kU; ++u)
                if (u < nvalid) store_pair<TG>(gp + u * sg, g[u][0], g[u][1], vec_out, ok0, ok1, accumulate);
        }
    }
    return pen;
}

template <typename TG, bool GRAD, bool HIST>
__global__ void __launch_bounds__(kTailThreads, kCtasPerSm) chan_tail_kernel(const ChanArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TailSmem &sm = *reinterpret_cast<TailSmem *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_strips = (int)((a.cols + kChanStrip - 1) / kChanStrip);
    const int n_items = n_strips * a.n_slices;
    const uint32_t flip = a.lambda < 0.0 ? 0x80000000u : 0u;

    // count window: the symbols [-kSymWin/2, kSymWin/2) that the clamp leaves alone
    const int32_t wlo = (int32_t)max((int64_t)-kSymWin / 2, (int64_t)a.qmin);
    const int32_t whi = (int32_t)max((int64_t)wlo, min((int64_t)kSymWin / 2, (int64_t)a.qmax + 1));
    const float inv = (float)(1.0 / (double)a.step);
    if (tid == 0) {
        sm.cc.inv = inv; sm.cc.wlo = wlo; sm.cc.whi = whi; sm.cc.qmin = a.qmin; sm.cc.qmax = a.qmax;
        sm.cc.flip = flip; sm.cc.hist = reinterpret_cast<unsigned long long *>(a.hist);
    }

    ChanLane ln;
    ln.a_addr = (uint32_t)__cvta_generic_to_shared(&sm.a1[0][0][lane]);
    ln.b_addr = (uint32_t)__cvta_generic_to_shared(&sm.bt[0][0][lane]);
    ln.e_lo = 1u;
    ln.inv = inv;
    ln.t_lo = (float)wlo - 0.5f;
    ln.t_hi = (float)whi;
    // |t| below min(-wlo, whi) is inside the window for sure; one compare per block of rows finds the rest
    ln.near = (wlo < 0 && whi > 0) ? (float)min(-wlo, whi) : 0.0f;
    // floor(tc) lies in [wlo - 1, whi]; cell = floor(tc) - (wlo - 1)
    ln.cnt_off = (uint32_t)__cvta_generic_to_shared(sm.cnt) - (kMagicBits + (uint32_t)(wlo - 1)) * 4u;
    ln.cnt_addr = (uint32_t)__cvta_generic_to_shared(sm.cnt);
    ln.cbase = 0x8000u;

    if constexpr (HIST) {
        for (int i = tid; i < kSymWin + 4; i += kTailThreads) sm.cnt[i] = 0u;
        for (int i = tid; i < kSlowWin; i += kTailThreads) sm.win[i] = 0u;
        if (tid < 2) sm.clampc[tid] = 0u;
    }
    const bool vec_in = ((reinterpret_cast<uintptr_t>(a.x) & 3u) == 0) && ((a.ld & 1) == 0) && ((a.cols & 1) == 0);
    const bool vec_out = ((reinterpret_cast<uintptr_t>(a.grad) & (2 * sizeof(TG) - 1)) == 0) && ((a.grad_ld & 1) == 0) &&
                         ((a.cols & 1) == 0);
    const bool accumulate = a.accumulate != 0;
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(&sm.ring[0][0][tid]);
    int cur_strip = -1;
    bool sym_pending = false;      // symbol cells hold counts that are not in the histogram yet
    __syncthreads();

    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        // neighbouring CTAs take neighbouring strips of the same rows: their row pieces are adjacent in memory
        const int strip = item % n_strips, slice = item / n_strips;
        // slices are cut at multiples of the rows one pass of the CTA covers, so that only the last one is ragged
        constexpr int64_t kPass = (int64_t)kTailWarps * kU;
        const int64_t n_pass = (a.rows + kPass - 1) / kPass;
        const int64_t r_begin = n_pass * slice / a.n_slices * kPass;
        const int64_t r_end = min(a.rows, n_pass * (slice + 1) / a.n_slices * kPass);
        const int64_t c0 = (int64_t)strip * kChanStrip + 2 * lane;
        const bool ok0 = c0 < a.cols, ok1 = c0 + 1 < a.cols;

        if (GRAD && strip != cur_strip) {
            // ---- the tables of this strip's 64 columns, built once per strip by chan_tables_kernel
            cur_strip = strip;
            __syncthreads();
            const uint4 *src = reinterpret_cast<const uint4 *>(a.tab + (int64_t)strip * kTabFloats);
            uint4 *dst = reinterpret_cast<uint4 *>(&sm.a1[0][0][0]);      // a1 and bt are contiguous
            for (int i = tid; i < kTabFloats / 4; i += kTailThreads) dst[i] = __ldg(src + i);
            if (tid < kChanStrip) {
                const int64_t c = (int64_t)strip * kChanStrip + tid;
                const bool ok = c < a.cols;
                sm.colL[tid] = ok ? a.L[c] : __longlong_as_double(0x7FF8000000000000ll);
                sm.colb[tid] = ok ? a.b[c] : 0.0;
            }
            ln.e_lo = (uint32_t)__ldg(a.tab_elo + strip);
            __syncthreads();
        }

        // ---- how this item counts: by symbol if the symbol window holds the bulk of the strip's symbols, else by
        // bit pattern over the 16 binades up to the strip's largest magnitude (quantised when flushed)
        bool pat = false;
        if constexpr (HIST) {
            __syncthreads();
            if (tid == 0) { sm.amax_bits = 0; sm.sd_bits = 0; }
            __syncthreads();
            if (tid < kChanStrip && (int64_t)strip * kChanStrip + tid < a.cols) {
                atomicMax(&sm.amax_bits, (int)__float_as_uint(a.amax[(int64_t)strip * kChanStrip + tid]));
                atomicMax(&sm.sd_bits, (int)__float_as_uint(a.sd[(int64_t)strip * kChanStrip + tid]));
            }
            __syncthreads();
            // by symbol while the window reaches 6.5 standard deviations of the widest column (the few symbols
            // beyond are counted one by one)
            pat = !(6.5f * __int_as_float(sm.sd_bits) * inv < ln.near);
            if (pat) {
                if (sym_pending) { chan_flush(sm, false, 0u, a); sym_pending = false; }
                // 16 binades ending one above that of the largest magnitude (that last one is empty, so no element
                // has the first pattern after the window), or ending at the top binade of the format
                const int e_top = sm.amax_bits >> 23;
                const int e_hi = e_top >= 253 ? 255 : max(16, e_top + 1);
                ln.cbase = (uint32_t)(e_hi - 15) << 7;
            } else {
                sym_pending = true;
            }
        }

        // ---- stream the rows of the slice: warp w takes rows r_begin + w, + kTailWarps, ...
        double pen[2] = {0.0, 0.0};
        auto stream_item = [&](auto pat_tag) {
            constexpr bool PAT = decltype(pat_tag)::value;
            const int64_t r0 = r_begin + warp;
            int n_mine = r0 < r_end ? (int)((r_end - r0 + kTailWarps - 1) / kTailWarps) : 0;      // rows of this warp
            const int64_t sin = (int64_t)kTailWarps * a.ld, sg = (int64_t)kTailWarps * a.grad_ld;
            const uint16_t *p = a.x + c0 + r0 * a.ld;
            TG *gp = GRAD && a.grad != nullptr ? reinterpret_cast<TG *>(a.grad) + c0 + r0 * a.grad_ld : nullptr;
            // Whole blocks of a whole strip with aligned rows: each thread stages its words of the next block
            // in its own ring slots with asynchronous copies while it works on the current one (one commit
            // group per block, so the group that must have landed is always the one before the last).
            if ((int64_t)strip * kChanStrip + kChanStrip <= a.cols && vec_in && (gp == nullptr || vec_out) && !accumulate) {
                const int n_blocks = n_mine / kU;
                auto stage = [&](const uint16_t *src, uint32_t dst) {
#pragma unroll
                    for (int u = 0; u < kU; ++u)
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst + (uint32_t)u * kRowBytes), "l"(src + u * sin) : "memory");
                };
                if (n_blocks > 0) stage(p, ring);
                asm volatile("cp.async.commit_group;" ::: "memory");
                for (int bk = 0; bk < n_blocks; ++bk) {
                    const uint32_t cur = ring + (uint32_t)(bk & 1) * kU * kRowBytes;
                    if (bk + 1 < n_blocks) stage(p + kU * sin, ring + (uint32_t)((bk + 1) & 1) * kU * kRowBytes);
                    asm volatile("cp.async.commit_group;" ::: "memory");
                    asm volatile("cp.async.wait_group 1;" ::: "memory");
                    chan_block_fast<TG, GRAD, HIST, PAT>(cur, gp, sg, lane, ln, sm, pen);
                    p += kU * sin;
                    if (gp != nullptr) gp += kU * sg;
                }
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                n_mine -= n_blocks * kU;
            }
            for (; n_mine > 0; n_mine -= kU, p += kU * sin, gp += gp != nullptr ? kU * sg : 0) {
                const double2 d = chan_block_guarded<TG, GRAD, HIST, PAT>(p, sin, gp, sg, min(n_mine, kU), ok0, ok1, vec_in,
                                                                          vec_out, accumulate, lane, ln, &sm);
                pen[0] += d.x;
                pen[1] += d.y;
            }
        };
        if (HIST && pat) stream_item(std::true_type{});
        else stream_item(std::false_type{});
        if constexpr (HIST) {
            if (pat) {           // the window moves with the strip: empty it now
                __syncthreads();
                chan_flush(sm, true, ln.cbase, a);
            }
        }

        if constexpr (GRAD) {
            // penalty partial of every column of the strip: the warps in a fixed order
            sm.red[warp][2 * lane] = pen[0];
            sm.red[warp][2 * lane + 1] = pen[1];
            __syncthreads();
            if (tid < kChanStrip) {
                const int64_t c = (int64_t)strip * kChanStrip + tid;
                if (c < a.cols) {
                    double ps = 0.0;
                    for (int wv = 0; wv < kTailWarps; ++wv) ps += sm.red[wv][tid];
                    a.pen[(int64_t)slice * a.cols + c] = ps;
                }
            }
            __syncthreads();
        }
    }

    if constexpr (HIST) {
        __syncthreads();
        if (sym_pending) chan_flush(sm, false, 0u, a);
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
    chan_fit_kernel<<<(unsigned)((a.cols + kFitCols - 1) / kFitCols), kFitCols * kFitGroups, 0, st>>>(a);
    return cudaGetLastError();
}

// Row slices per strip: enough items to fill two CTAs per SM, in whole rounds of the grid where
// there are more items than CTAs, and at least 512 rows per item so that the tables (192 entries
// per column) stay cheap next to the rows they serve.
int chan_slices(int64_t rows, int64_t cols, int sm_count, int strip)
{
    const int64_t n_strips = (cols + strip - 1) / strip;
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
    if (a.do_grad) {
        chan_tables_kernel<<<(unsigned)((a.cols + kChanStrip - 1) / kChanStrip), kTailThreads, 0, st>>>(a);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
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
