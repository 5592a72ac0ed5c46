// bf16-input sweep with a gradient and/or a histogram (optionally the moments too), specialised
// for the fact that a bf16 value is one of 65536 bit patterns.
//
// Persistent CTAs each walk one contiguous range of tiles.  Inside a segment that range is one
// contiguous run of elements, streamed as 128-bit vectors.
//   * gradient: |g| depends only on the 15-bit magnitude pattern.  |g| = A[e] * B[j] with e the
//     exponent field and j the 7 mantissa bits: A[e] = 2^(L + b (e-127)), B[j] = (1 + j/128)^b,
//     both rounded once from fp64, so the product is within 1.5 ulp for every shape beta.
//   * histogram: elements are counted in shared memory, by quantised symbol when the quantiser is
//     coarse and by bit pattern otherwise; patterns become symbols only when the table is flushed,
//     i.e. when the histogram, its step or the window changes, or the CTA ends.  Counts are
//     integers, so every order of additions gives the same table.
// The kernel's limits are instruction issue and the shared-memory pipe (one 128-byte wavefront per
// clock and SM), so the element path is kept to two table reads, one atomic and about twenty
// instructions, with tables laid out against bank conflicts:
//   * A is indexed by the exponent field: the lanes of a warp hold a handful of neighbouring
//     exponents, which fall in different banks or in the same word.  B is indexed by the random
//     mantissa bits and is therefore replicated once per bank (lane l reads word l of row j).
//     Exponents whose A cannot be a single normal fp32 factor (zero/subnormal, inf/nan, far
//     binades) hold NaN; the NaN reaches the penalty partial of the vector, whose range check
//     then sends the vector to the exact path.
//   * counts have two layouts.  Symbol mode, used when symbols [-192, 192) hold all but the far
//     tails (192 steps >= 6.5 standard deviations): one row of 32 words per symbol, lane l counts
//     in word l; the symbol is floor(x * inv) taken with a round-down add of 1.5 * 2^23.  Pattern
//     mode otherwise: one cell per bf16 magnitude pattern and sign over 16 binades below 2^5
//     standard deviations, two replicas per cell selected by the lowest lane bit.
//     An element outside the count window (a far-tail symbol, a tiny or huge pattern, inf, nan)
//     counts in a sentinel cell and is redone after its vector.
// Input vectors reach each thread through a private ring of shared-memory slots filled by
// asynchronous copies issued kDepth iterations ahead: bytes in flight cost no registers.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <float.h>

#include "gg_device.cuh"
#include "gg_fit_table.cuh"
#include "gg_internal.h"

namespace gg {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kCtasPerSm = 2;
constexpr int kDepth = 4;                           // input vectors staged ahead per thread
constexpr int kCntBinades = 16;                     // pattern-count window
constexpr uint32_t kCntPat = kCntBinades * 128;     // magnitude patterns in it
constexpr int kRep = 2;                             // replicas of every pattern-count cell
constexpr uint32_t kSymCells = 384;                 // symbol-count window: symbols [-192, 192)
constexpr uint32_t kSymBase = kMagicBits - kSymCells / 2;
constexpr int kSymWin = 512;                        // secondary symbol window [-256, 256) of the rare path
constexpr uint32_t kCntWords = (kSymCells + 2) * 32 > (kCntPat + 1) * 2 * kRep ? (kSymCells + 2) * 32
                                                                              : (kCntPat + 1) * 2 * kRep;
enum : int { kModePattern = 1, kModeSymbol = 2 };

// Constants of the current segment / histogram that only the cold paths need: kept in shared
// memory so that the streaming loop does not carry them in registers.
struct Cold {
    double L, b;               // g = 2^(L + b log2|x|)
    uint32_t sign_flip;        // 0x80000000 if lambda < 0 (the tables then hold -|g|)
    int active;                // 0: the gradient is zero everywhere
    float inv;                 // quantiser: q = floor(x * inv)
    int32_t qmin, qmax;
    unsigned long long *row;   // the current histogram, bin 0 = symbol qmin
    uint32_t c_base;           // first magnitude pattern of the pattern-count window
    int symbol_mode;           // layout of cnt: 1 = rows of symbols, 0 = cells of patterns
    float eg_c;                // code-length gradient (kEg): the factor c of the segment
    uint32_t eg_two_k;
};

struct ClusterPart {
    double s1, s2;
    uint32_t bad;
    float mn, mx;
};

struct Smem {
    // pattern mode: cell ((p * 2 + sign) * kRep + r) = magnitude pattern c_base + p, replica r; slot
    // p = kCntPat is the sentinel that swallows the counts of out-of-window elements.
    // symbol mode: word ((s + 1) * 32 + lane) = symbol s - kSymCells/2 counted by that lane; the rows
    // before and after the window (s = -1 and s = kSymCells) are the sentinels of the two tails.
    uint32_t cnt[kCntWords];
    float brep[128 * 32];            // row j: B[j] in every bank
    float2 A[256];                   // every exponent: value = A.x * A.y, A.y a power of two
    float B[128];
    double lg[128];                  // log2(1 + j/128)
    uint32_t win[kSymWin];
    double red[3][kWarps];
    uint32_t bad[kWarps];
    float mn[kWarps], mx[kWarps];
    uint32_t clampc[2];
    Cold cold;
    int e_top;
    // one-cluster-per-segment kernel: this CTA's moments of the current segment (two slots, used in turn: the other
    // CTAs of the cluster read them) and the barrier its bulk copies complete on
    ClusterPart cpart[2];
    alignas(8) unsigned long long mbar;
    // per-thread ring of input vectors in flight; the one-cluster-per-segment kernel keeps its share of the segment
    // here and in the dynamic shared memory that follows the structure
    alignas(128) uint4 stage[kDepth][kThreads];
};

// A[e] as one factor (with lambda's sign), NaN where that is not possible.  Static shared memory:
// its address is a compile-time constant, so a look-up is an index and a load.
__shared__ float s_a1[256];

// |g| (with lambda's sign) for a magnitude pattern the A/B tables do not cover: zero, subnormal,
// inf, nan.
__device__ __noinline__ float grad_rare(uint32_t mag, const Smem &sm)
{
    const float ax = __uint_as_float(mag << 16);
    if (!sm.cold.active || ax == 0.0f) return 0.0f;
    const float v = (float)exp2(sm.cold.L + sm.cold.b * log2((double)ax));
    return __uint_as_float(__float_as_uint(v) ^ sm.cold.sign_flip);
}

// The gradient of any magnitude pattern from the two-factor tables (exact path).
__device__ __noinline__ float grad_exact(uint32_t mag, const Smem &sm)
{
    const uint32_t e = mag >> 7;
    if (e - 1u < 254u) {
        const float2 a = sm.A[e];
        return (a.x * sm.B[mag & 127u]) * a.y;
    }
    return grad_rare(mag, sm);
}

// Quantises one value and adds n to its symbol's count: the shared symbol window when allowed and
// in reach, else global memory.
__device__ __forceinline__ void count_symbol(float x, uint32_t n, bool use_window, Smem &sm)
{
    const float t = __fmul_rn(x, sm.cold.inv);
    if (t == t) {                                  // NaN is skipped
        int q = __float2int_rd(t);                 // floor, saturating
        const int qmin = sm.cold.qmin, qmax = sm.cold.qmax;
        if (q < qmin) { q = qmin; atomicAdd(&sm.clampc[0], n); }
        else if (q > qmax) { q = qmax; atomicAdd(&sm.clampc[1], n); }
        const uint32_t w = (uint32_t)(q + kSymWin / 2);
        if (use_window && w < (uint32_t)kSymWin) atomicAdd(&sm.win[w], n);
        else atomicAdd(&sm.cold.row[q - qmin], (unsigned long long)n);
    }
}

__device__ __noinline__ void count_rare(uint32_t xb, Smem &sm) { count_symbol(__uint_as_float(xb), 1u, true, sm); }

struct Acc {
    double s1 = 0.0, s2 = 0.0, pen = 0.0;
    uint32_t bad = 0;
    float xmin = INFINITY, xmax = -INFINITY;     // extremes of the elements taken one by one
    // extremes of the elements taken as vectors: two bf16 lanes (even and odd elements)
    __nv_bfloat162 mn2 = __floats2bfloat162_rn(INFINITY, INFINITY), mx2 = __floats2bfloat162_rn(-INFINITY, -INFINITY);
};

struct Run {   // fp32 partials of one short run of elements
    float m1 = 0.0f, m2 = 0.0f, mp = 0.0f;
    // penalty terms of elements taken two at a time: sums of x * g (= lambda's sign times |x| |g|), even and odd
    // elements side by side in one 64-bit register
    uint64_t mp2 = 0ull;
};

// Two fp32 numbers in one 64-bit register, and the sm_100 arithmetic on such pairs (one instruction for both).
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2_rd(uint64_t a, uint64_t b)      // both sums rounded down
{
    uint64_t d;
    asm("add.rm.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// The fp32 penalty partial of a run: elements taken one by one plus the pairs (whose sums carry lambda's sign).
__device__ __forceinline__ float run_penalty(const Run &r)
{
    float lo, hi;
    unpack2(r.mp2, lo, hi);
    return r.mp + fabsf(lo + hi);
}

// Per-thread constants of the element path.
struct Lane {
    uint32_t cbase;    // first magnitude pattern of the pattern-count window
    // 32-bit shared-memory addresses of this lane's word in the first row of each table
    uint32_t b_addr;   // brep + lane * 4
    uint32_t s_addr;   // symbol mode: row of symbol -kSymCells/2 in cnt, + lane * 4
    uint32_t p_addr;   // pattern mode: cnt + (lane mod kRep) * 4
    float inv;         // quantiser scale (symbol mode)
    uint64_t inv2;     // the same twice, for the pair arithmetic
    float eg_c;        // code-length gradient (kEg): c of the segment, 2^k, the clamp of the symbols
    uint32_t eg_two_k;
    int32_t qmin, qmax;
};

template <int FLAGS>
__device__ __forceinline__ void moments_elem(uint32_t xb, Acc &acc, Run &r)
{
    if constexpr ((FLAGS & kMoments) != 0) {
        const uint32_t am = xb & 0x7FFFFFFFu;
        const bool fin = am < 0x7F800000u;
        const float af = fin ? __uint_as_float(am) : 0.0f;
        r.m1 += af;
        r.m2 = fmaf(af, af, r.m2);
        acc.bad += fin ? 0u : 1u;
        acc.xmin = fminf(acc.xmin, __uint_as_float(xb));     // fminf / fmaxf return the non-NaN operand
        acc.xmax = fmaxf(acc.xmax, __uint_as_float(xb));
    }
}

// Row of a value in the symbol-count table: floor(x * inv) + kSymCells/2 as an unsigned number, so
// that every symbol outside the window, and inf and nan, give a row >= kSymCells.
__device__ __forceinline__ uint32_t symbol_row(uint32_t xb, float inv)
{
    const float t = __fmul_rn(__uint_as_float(xb), inv);
    // for |t| < 2^22 the sum lies in [2^23, 2^24) where floats are the integers: rounding down gives floor
    return __float_as_uint(__fadd_rd(t, __uint_as_float(kMagicBits))) - kSymBase;
}

// One element of a 32-bit word w holding two bf16 values: HALF 0 is the low half, 1 the high half.
// Branch free.  Gradient: a NaN entry of s_a1 (an exponent outside the single-factor range) makes
// the vector's penalty partial NaN, which the caller checks once per vector.  Count: `anyc` keeps
// the largest |x * inv| (symbol mode) or window index (pattern mode) so that one compare per
// vector finds elements that missed the window; those count in the sentinel cells.
template <int FLAGS, int MODE, int HALF, bool MOMENTS_HERE = true>
__device__ __forceinline__ float one_elem(uint32_t w, const Lane &ln, Acc &acc, Run &r, uint32_t &anyc)
{
    const uint32_t xb = HALF ? (w & 0xFFFF0000u) : (w << 16);     // the value as fp32 bits
    if constexpr (MOMENTS_HERE) moments_elem<FLAGS>(xb, acc, r);
    float ga = 0.0f;
    constexpr bool EG = (FLAGS & kEg) != 0;
    if constexpr ((FLAGS & kGrad) != 0 && !EG) {
        const uint32_t e4 = HALF ? ((w >> 21) & 0x3FCu) : ((w >> 5) & 0x3FCu);     // exponent field * 4
        const uint32_t j = HALF ? ((w >> 16) & 127u) : (w & 127u);
        const float a = *reinterpret_cast<const float *>(reinterpret_cast<const char *>(s_a1) + e4);
        ga = a * lds_f32(j * 128u + ln.b_addr);
    }
    if constexpr (EG && MODE != kModeSymbol) {
        // (pattern counting does not form the symbol: the quantiser here; a nan gives no gradient)
        const float t = __fmul_rn(__uint_as_float(xb), ln.inv);
        const int q = max(ln.qmin, min(ln.qmax, __float2int_rd(t)));
        ga = (t == t) ? eg_grad_of_symbol(q, ln.eg_c, ln.eg_two_k) : 0.0f;
    }
    if constexpr ((FLAGS & kHist) != 0) {
        if constexpr (MODE == kModeSymbol) {
            // t clamped to just outside the window: the floor of the clamped value lands on a sentinel
            // row for either tail (and for nan, which the maximum replaces by the lower bound)
            const float t = __fmul_rn(__uint_as_float(xb), ln.inv);
            // (one float maximum with an absolute-value operand; a nan is ignored here, which is right: it lands on
            // a sentinel row and is not to be counted)
            // (with the code-length gradient a nan must be found too, since its gradient is zero and not the sentinel
            // row's: the maximum is then taken on the bit patterns, where a nan is the largest)
            if constexpr (EG) anyc = max(anyc, __float_as_uint(fabsf(t)));
            else anyc = __float_as_uint(fmaxf(__uint_as_float(anyc), fabsf(t)));
            const float tc = fminf(fmaxf(t, -(float)(kSymCells / 2) - 0.5f), (float)(kSymCells / 2));
            // for |t| < 2^22 the sum lies in [2^23, 2^24) where floats are the integers: rounding down gives floor
            const uint32_t fb = __float_as_uint(__fadd_rd(tc, __uint_as_float(kMagicBits)));
            red_inc(fb * 128u + ln.s_addr);     // (s_addr already holds minus 128 times the bits of symbol -kSymCells/2)
            // (the symbols of the window are not clamped in this mode; an element outside it is redone by fix_elem)
            if constexpr (EG) ga = eg_grad_of_symbol((int)(fb - kMagicBits), ln.eg_c, ln.eg_two_k);
        } else {
            static_assert(kRep == 2, "cell stride");
            const uint32_t mag = HALF ? ((w >> 16) & 0x7FFFu) : (w & 0x7FFFu);
            uint32_t p = mag - ln.cbase;
            anyc = max(anyc, p);
            p = min(p, kCntPat);
            const uint32_t sign8 = HALF ? ((w >> 28) & 8u) : ((w >> 12) & 8u);
            red_inc(p * 16u + sign8 + ln.p_addr);
        }
    }
    if constexpr (EG) {
        // (no penalty partial: the rate comes from the histogram; zero has no gradient)
        ga = (xb << 1) != 0u ? ga : 0.0f;
        return __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));
    } else if constexpr ((FLAGS & kGrad) != 0) {
        r.mp = fmaf(fabsf(__uint_as_float(xb)), fabsf(ga), r.mp);
        return __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));   // the table carries lambda's sign
    }
    return 0.0f;
}

// The two elements of a 32-bit word at once, with the pair arithmetic of sm_100 where two elements do the same
// thing: the table product, the penalty term, the quantiser scaling and the round-down add that takes the floor.
// Same results as two calls of one_elem, element by element.
template <int FLAGS, int MODE>
__device__ __forceinline__ void two_elems(uint32_t w, const Lane &ln, Run &r, uint32_t &anyc, float &g_lo, float &g_hi)
{
    const uint32_t xlo = w << 16, xhi = w & 0xFFFF0000u;
    const uint64_t xx = pack2(__uint_as_float(xlo), __uint_as_float(xhi));
    g_lo = 0.0f;
    g_hi = 0.0f;
    if constexpr ((FLAGS & kGrad) != 0) {
        const float alo = *reinterpret_cast<const float *>(reinterpret_cast<const char *>(s_a1) + ((w >> 5) & 0x3FCu));
        const float ahi = *reinterpret_cast<const float *>(reinterpret_cast<const char *>(s_a1) + ((w >> 21) & 0x3FCu));
        const float blo = lds_f32((w & 127u) * 128u + ln.b_addr), bhi = lds_f32(((w >> 16) & 127u) * 128u + ln.b_addr);
        float ga_lo, ga_hi;
        unpack2(mul2(pack2(alo, ahi), pack2(blo, bhi)), ga_lo, ga_hi);
        g_lo = __uint_as_float(__float_as_uint(ga_lo) ^ (xlo & 0x80000000u));   // the table carries lambda's sign
        g_hi = __uint_as_float(__float_as_uint(ga_hi) ^ (xhi & 0x80000000u));
        r.mp2 = fma2(xx, pack2(g_lo, g_hi), r.mp2);
    }
    if constexpr ((FLAGS & kHist) != 0) {
        if constexpr (MODE == kModeSymbol) {
            float t_lo, t_hi;
            unpack2(mul2(xx, ln.inv2), t_lo, t_hi);
            anyc = __float_as_uint(fmaxf(__uint_as_float(anyc), fmaxf(fabsf(t_lo), fabsf(t_hi))));
            const float c_lo = fminf(fmaxf(t_lo, -(float)(kSymCells / 2) - 0.5f), (float)(kSymCells / 2));
            const float c_hi = fminf(fmaxf(t_hi, -(float)(kSymCells / 2) - 0.5f), (float)(kSymCells / 2));
            float f_lo, f_hi;
            unpack2(add2_rd(pack2(c_lo, c_hi), pack2(__uint_as_float(kMagicBits), __uint_as_float(kMagicBits))), f_lo, f_hi);
            red_inc(__float_as_uint(f_lo) * 128u + ln.s_addr);
            red_inc(__float_as_uint(f_hi) * 128u + ln.s_addr);
        } else {
            static_assert(kRep == 2, "cell stride");
            uint32_t p_lo = (w & 0x7FFFu) - ln.cbase, p_hi = ((w >> 16) & 0x7FFFu) - ln.cbase;
            anyc = max(anyc, max(p_lo, p_hi));
            p_lo = min(p_lo, kCntPat);
            p_hi = min(p_hi, kCntPat);
            red_inc(p_lo * 16u + ((w >> 12) & 8u) + ln.p_addr);
            red_inc(p_hi * 16u + ((w >> 28) & 8u) + ln.p_addr);
        }
    }
}

// (symbol mode: some |t| >= kSymCells/2, compared as bit patterns of non-negative floats; the exact
// test is redone per element by fix_elem)
template <int MODE>
__device__ __forceinline__ bool count_miss(uint32_t anyc)
{
    if constexpr (MODE == kModeSymbol) return anyc >= __float_as_uint((float)(kSymCells / 2));
    return anyc >= kCntPat;
}

// Redo of whatever part of an element (given as fp32 bits) the branch-free path could not do; g is
// the gradient from the first pass.  grad_bad: the vector's penalty partial left the fp32 range.
template <int FLAGS, int MODE>
__device__ __forceinline__ float fix_elem(uint32_t xb, float g, bool grad_bad, const Lane &ln, Smem &sm)
{
    const uint32_t mag = (xb & 0x7FFFFFFFu) >> 16;
    if constexpr ((FLAGS & kGrad) != 0 && (FLAGS & kEg) == 0) {
        if (grad_bad) {
            const float a = s_a1[mag >> 7];
            if (a != a) {     // this element read a NaN marker: zero needs no table, the rest the exact path
                const float ga = mag == 0u ? 0.0f : grad_exact(mag, sm);
                g = __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));
            }
        }
    }
    if constexpr ((FLAGS & kHist) != 0) {
        bool miss;
        if constexpr (MODE == kModeSymbol) miss = symbol_row(xb, ln.inv) >= kSymCells;
        else miss = mag - ln.cbase >= kCntPat;
        if (miss) count_rare(xb, sm);
        if constexpr ((FLAGS & kEg) != 0) {
            // (symbol mode: the element missed the window, so its symbol was a sentinel's)
            if (miss && MODE == kModeSymbol) g = eg_grad_exact(xb, ln.inv, ln.qmin, ln.qmax, ln.eg_c, ln.eg_two_k);
        }
    }
    return g;
}

// fp64 penalty terms |x| |g| of up to eight patterns packed in four words (rare path).
__device__ __noinline__ double pen_rare(uint4 raw, int n, const Smem &sm)
{
    if (!sm.cold.active) return 0.0;
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    double dp = 0.0;
    for (int e = 0; e < n; ++e) {
        const uint32_t h = (w[e >> 1] >> ((e & 1) * 16)) & 0x7FFFu;
        const double ax = (double)__uint_as_float(h << 16);
        if (ax != 0.0) dp += ax * exp2(sm.cold.L + sm.cold.b * log2(ax));
    }
    return dp;
}

template <int FLAGS>
__device__ __forceinline__ void close_run(const uint4 &raw, int n, Run &r, Acc &acc, const Smem &sm)
{
    if constexpr ((FLAGS & kMoments) != 0) {
        if (run_sums_exact_enough(r.m1, r.m2)) {
            acc.s1 += (double)r.m1;
            acc.s2 += (double)r.m2;
        } else {     // a square or a sum outside the fp32 range: this run again in fp64
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
            for (int e = 0; e < n; ++e) {
                const uint32_t h = (w[e >> 1] >> ((e & 1) * 16)) & 0x7FFFu;
                if (h < 0x7F80u) {
                    const double ax = (double)__uint_as_float(h << 16);
                    acc.s1 += ax;
                    acc.s2 += ax * ax;
                } else {
                    acc.bad += 1u;     // (elements taken one by one never get here with an inf or nan: they count it themselves)
                }
            }
        }
    }
    if constexpr ((FLAGS & kGrad) != 0 && (FLAGS & kEg) == 0) {
        // a product or a gradient that left the fp32 range, or a NaN marker, sends the run to fp64
        if (run_penalty(r) <= FLT_MAX) acc.pen += (double)run_penalty(r);
        else acc.pen += pen_rare(raw, n, sm);
    }
}

// Eight gradient values to g.  `wide`: g is 32-byte aligned, so fp32 output goes out as one
// 256-bit store per thread (a full 32-byte sector per lane, 1 KB contiguous per warp).
template <typename TG>
__device__ __forceinline__ void store8(TG *g, const float (&v)[8], bool accumulate, bool wide)
{
    if constexpr (sizeof(TG) == 4) {
        if (wide && !accumulate) {
            // written once, never re-read by this pass: streaming (evict-first) store
            asm volatile("st.global.cs.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(g), "f"(v[0]), "f"(v[1]),
                         "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
                         : "memory");
            return;
        }
        float4 *p = reinterpret_cast<float4 *>(g);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            float4 o = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            if (accumulate) {
                const float4 old = p[i];
                o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
            }
            __stcs(p + i, o);
        }
    } else {
        uint32_t w[4];
        const uint32_t *p = reinterpret_cast<const uint32_t *>(g);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float lo = v[2 * i], hi = v[2 * i + 1];
            if (accumulate) {
                const uint32_t old = p[i];
                lo += __uint_as_float(old << 16);
                hi += __uint_as_float(old & 0xFFFF0000u);
            }
            w[i] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) |
                   ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
        }
        __stcs(reinterpret_cast<uint4 *>(g), make_uint4(w[0], w[1], w[2], w[3]));
    }
}

// Exponent field of the top binade of the pattern-count window: the binade of 2^above times `scale`.
__device__ __forceinline__ int window_top_exponent(double scale, int above)
{
    int e = 127 + above;
    if (scale > 0.0 && scale < 1e300) e = ilogb(scale) + 127 + above;
    return max(kCntBinades, min(254, e));
}

// Adds the counted cells to the current histogram and empties the tables.
__device__ void flush_counts(Smem &sm, uint64_t *clamped, int hid)
{
    // (callers synchronise before: all counting under the old key is complete)
    if (sm.cold.symbol_mode) {
        const int lane = threadIdx.x & 31;
        // (every CTA starts at another row / cell: CTAs that flush into one histogram at the same time
        // would otherwise walk its addresses in step and serialise on them)
        for (uint32_t r0 = threadIdx.x >> 5; r0 < kSymCells + 2; r0 += kWarps) {   // row 0 and the last: sentinels
            const uint32_t row = (r0 + blockIdx.x * 13u) % (kSymCells + 2);
            const uint32_t v = sm.cnt[row * 32 + lane];
            const uint32_t n = __reduce_add_sync(0xFFFFFFFFu, v);
            if (n != 0u) {
                sm.cnt[row * 32 + lane] = 0u;
                // the window's symbols lie inside [qmin, qmax] in this mode; the sentinel rows are only emptied
                if (lane == 0 && row >= 1 && row <= kSymCells)
                    atomicAdd(&sm.cold.row[((int)row - 1 - (int)(kSymCells / 2)) - sm.cold.qmin], (unsigned long long)n);
            }
        }
    } else {
        const uint32_t c_base = sm.cold.c_base;
        for (uint32_t i = threadIdx.x; i < (kCntPat + 1) * 2; i += kThreads) {
            const uint32_t c = (i + blockIdx.x * 61u) % ((kCntPat + 1) * 2);     // c = p * 2 + sign
            uint2 *cell = reinterpret_cast<uint2 *>(sm.cnt) + c;
            const uint2 v = *cell;
            const uint32_t n = v.x + v.y;
            if (n != 0u) {
                *cell = make_uint2(0u, 0u);
                if (c < kCntPat * 2) {          // the sentinel slot is only emptied
                    const uint32_t h = (c_base + (c >> 1)) | ((c & 1u) << 15);
                    count_symbol(__uint_as_float(h << 16), n, false, sm);
                }
            }
        }
    }
    for (int i = threadIdx.x; i < kSymWin; i += kThreads) {
        const uint32_t n = sm.win[i];
        if (n != 0u) {
            sm.win[i] = 0u;
            atomicAdd(&sm.cold.row[(i - kSymWin / 2) - sm.cold.qmin], (unsigned long long)n);
        }
    }
    __syncthreads();
    if (threadIdx.x < 2) {
        const uint32_t n = sm.clampc[threadIdx.x];
        if (n != 0u && clamped != nullptr)
            atomicAdd(reinterpret_cast<unsigned long long *>(clamped) + 2 * hid + threadIdx.x, (unsigned long long)n);
        sm.clampc[threadIdx.x] = 0u;
    }
    __syncthreads();
}

template <int FLAGS>
__device__ __forceinline__ void zero_partials(const TileScratch &part, int t)
{
    if constexpr ((FLAGS & kMoments) != 0) {
        part.s1[t] = 0.0; part.s2[t] = 0.0; part.bad[t] = 0u;
        part.xmin[t] = INFINITY; part.xmax[t] = -INFINITY;
    }
    if constexpr ((FLAGS & kGrad) != 0) part.pen[t] = 0.0;
}

// Block reduction in a fixed order (butterfly inside each warp, then the warps in sequence) of the
// partial sums of one run of tiles [t0, t1); the result goes to the slot of t0, zeros to the rest.
template <int FLAGS>
__device__ void reduce_partials(const TileScratch &part, int t0, int t1, const Acc &acc, Smem &sm)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if constexpr ((FLAGS & kMoments) != 0) {
        const double w1 = warp_sum(acc.s1), w2 = warp_sum(acc.s2);
        const uint32_t wb = __reduce_add_sync(0xFFFFFFFFu, acc.bad);
        float wmin = fminf(acc.xmin, fminf(__low2float(acc.mn2), __high2float(acc.mn2)));
        float wmax = fmaxf(acc.xmax, fmaxf(__low2float(acc.mx2), __high2float(acc.mx2)));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            wmin = fminf(wmin, __shfl_xor_sync(0xFFFFFFFFu, wmin, o));
            wmax = fmaxf(wmax, __shfl_xor_sync(0xFFFFFFFFu, wmax, o));
        }
        if (lane == 0) {
            sm.red[0][warp] = w1; sm.red[1][warp] = w2; sm.bad[warp] = wb;
            sm.mn[warp] = wmin; sm.mx[warp] = wmax;
        }
    }
    if constexpr ((FLAGS & kGrad) != 0) {
        const double wp = warp_sum(acc.pen);
        if (lane == 0) sm.red[2][warp] = wp;
    }
    __syncthreads();
    for (int t = t0 + 1 + tid; t < t1; t += kThreads) zero_partials<FLAGS>(part, t);
    if (tid == 0) {
        if constexpr ((FLAGS & kMoments) != 0) {
            double r1 = 0.0, r2 = 0.0;
            uint32_t rb = 0;
            float rmin = INFINITY, rmax = -INFINITY;
            for (int w = 0; w < kWarps; ++w) {
                r1 += sm.red[0][w]; r2 += sm.red[1][w]; rb += sm.bad[w];
                rmin = fminf(rmin, sm.mn[w]); rmax = fmaxf(rmax, sm.mx[w]);
            }
            part.s1[t0] = r1; part.s2[t0] = r2; part.bad[t0] = rb;
            part.xmin[t0] = rmin; part.xmax[t0] = rmax;
        }
        if constexpr ((FLAGS & kGrad) != 0) {
            double rp = 0.0;
            for (int w = 0; w < kWarps; ++w) rp += sm.red[2][w];
            part.pen[t0] = sm.cold.sign_flip ? -rp : rp;     // the penalty carries lambda's sign
        }
    }
    __syncthreads();
}


template <typename TG, int FLAGS, int MODE>
__device__ __forceinline__ void process_vec(const uint4 &raw, TG *gdst, bool accumulate, bool wide, const Lane &ln,
                                            Smem &sm, Acc &acc)
{
    constexpr bool GRAD = (FLAGS & kGrad) != 0, HIST = (FLAGS & kHist) != 0;
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    float g[8];
    Run r;
    uint32_t anyc = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if constexpr ((FLAGS & kMoments) != 0) {
            // both elements of the word at once; an inf or nan makes the run's sums inf or nan, and the run is
            // then summed again element by element (close_run), where it is counted and left out
            const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
            r.m1 += fabsf(lo);
            r.m1 += fabsf(hi);
            r.m2 = fmaf(lo, lo, r.m2);
            r.m2 = fmaf(hi, hi, r.m2);
            const __nv_bfloat162 pr = *reinterpret_cast<const __nv_bfloat162 *>(&w[i]);
            acc.mn2 = __hmin2(acc.mn2, pr);      // return the non-NaN operand, like fminf
            acc.mx2 = __hmax2(acc.mx2, pr);
        }
        // (the pair arithmetic saves a tenth of the instructions: a gain where instruction issue binds, which is the
        // bf16-gradient variant; with fp32 gradients the sweep is bound by DRAM and the board's power limit, and
        // measured 0.4 % slower with it)
        if constexpr (sizeof(TG) == 2 && (FLAGS & kEg) == 0) {
            two_elems<FLAGS, MODE>(w[i], ln, r, anyc, g[2 * i], g[2 * i + 1]);
        } else {
            g[2 * i] = one_elem<FLAGS, MODE, 0, false>(w[i], ln, acc, r, anyc);
            g[2 * i + 1] = one_elem<FLAGS, MODE, 1, false>(w[i], ln, acc, r, anyc);
        }
    }
    const bool grad_bad = GRAD && !(run_penalty(r) <= FLT_MAX);
    if (grad_bad || (HIST && count_miss<MODE>(anyc))) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t xb = (i & 1) ? (w[i >> 1] & 0xFFFF0000u) : (w[i >> 1] << 16);
            g[i] = fix_elem<FLAGS, MODE>(xb, g[i], grad_bad, ln, sm);
        }
    }
    close_run<FLAGS>(raw, 8, r, acc, sm);
    if constexpr (GRAD) {
        if (gdst != nullptr) store8<TG>(gdst, g, accumulate, wide);
    }
}

// One contiguous run of n elements: scalar head up to the first 16-byte boundary of x, 128-bit
// vector body fed through the asynchronous-copy ring, scalar tail.  If the gradient's address is
// not 16-byte aligned at the same element the whole run is scalar.
// One element taken by itself (the head and the tail of a run that do not fill a 16-byte vector).
template <typename TG, int FLAGS, int MODE>
__device__ __forceinline__ void scalar_elem(const uint16_t *x, TG *gout, int64_t idx, bool accumulate, const Lane &ln, Smem &sm, Acc &acc)
{
    constexpr bool GRAD = (FLAGS & kGrad) != 0, HIST = (FLAGS & kHist) != 0;
    const uint32_t h = (uint32_t)__ldg(x + idx);
    Run r;
    uint32_t anyc = 0;
    float g = one_elem<FLAGS, MODE, 0>(h, ln, acc, r, anyc);
    const bool grad_bad = GRAD && !(run_penalty(r) <= FLT_MAX);
    if (grad_bad || (HIST && count_miss<MODE>(anyc))) g = fix_elem<FLAGS, MODE>(h << 16, g, grad_bad, ln, sm);
    close_run<FLAGS>(make_uint4(h, 0u, 0u, 0u), 1, r, acc, sm);
    if constexpr (GRAD) {
        if (gout != nullptr) {
            float v = g;
            if constexpr (sizeof(TG) == 4) {
                if (accumulate) v += gout[idx];
                gout[idx] = v;
            } else {
                if (accumulate) v += __uint_as_float((uint32_t)gout[idx] << 16);
                gout[idx] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
            }
        }
    }
}

// L2 eviction hints of one run: vectors before `split` are copied with policy `first`, the others with `rest`.
struct Hints {
    uint64_t first = 0, rest = 0;
    int split = 0;
};

template <bool HINT>
__device__ __forceinline__ void copy16(uint32_t dst, const void *src, uint64_t policy)
{
    if constexpr (HINT)
        asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(policy) : "memory");
    else
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

template <typename TG, int FLAGS, int MODE, bool HINT = false>
__device__ __forceinline__ void process_range(const uint16_t *x, TG *gout, int64_t n, bool accumulate,
                                              const Lane &ln, Smem &sm, Acc &acc, const Hints hints = Hints())
{
    const int tid = threadIdx.x;
    int64_t head = (int64_t)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / 2u);
    head = min(head, n);
    if (gout != nullptr && (reinterpret_cast<uintptr_t>(gout + head) & 15u) != 0) head = n;
    // (the body starts a block of the gradient: 1 KB of fp32 or 512 bytes of bf16 per warp step; without a gradient, of x)
    else head = aligned_head(head, n, reinterpret_cast<uintptr_t>(x), reinterpret_cast<uintptr_t>(gout), 2u, (unsigned)sizeof(TG),
                             gout != nullptr ? 256u * (unsigned)sizeof(TG) : 512u);
    const int64_t nvec = (n - head) / 8;
    const int64_t tail0 = head + nvec * 8;

    for (int64_t i = tid; i < head + (n - tail0); i += kThreads) {
        const int64_t idx = i < head ? i : tail0 + (i - head);
        if (GG_IN_BOUNDS(idx, n)) scalar_elem<TG, FLAGS, MODE>(x, gout, idx, accumulate, ln, sm, acc);
    }

    // (a CTA's run never exceeds device memory / grid size elements: 32-bit vector indices suffice)
    // Each thread owns slot [d][tid] of every stage d: it fills them with asynchronous 16-byte
    // copies (one commit group per iteration, empty past the end so that the group count stays in
    // step) and reads a slot back once the group that filled it has landed.
    const uint4 *xv = reinterpret_cast<const uint4 *>(x + head) + tid;
    TG *gv = gout != nullptr ? gout + head + (int64_t)tid * 8 : nullptr;
    const bool wide = (reinterpret_cast<uintptr_t>(gv) & 31u) == 0;
    const int nv = (int)nvec;
    const uint32_t slot0 = (uint32_t)__cvta_generic_to_shared(&sm.stage[0][tid]);
    constexpr uint32_t kStageBytes = sizeof(uint4) * kThreads;
#pragma unroll
    for (int d = 0; d < kDepth - 1; ++d) {
        if (tid + d * kThreads < nv && GG_IN_BOUNDS(head + (int64_t)(tid + d * kThreads) * 8 + 7, n))
            copy16<HINT>(slot0 + d * kStageBytes, xv + d * kThreads, tid + d * kThreads < hints.split ? hints.first : hints.rest);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    // (the loop is unrolled over the stages, so that every slot is a compile-time offset)
    for (int v = tid; v < nv; v += kDepth * kThreads) {
#pragma unroll
        for (int d = 0; d < kDepth; ++d) {
            const int vd = v + d * kThreads;
            if (vd < nv) {
                // fill the slot emptied by the previous vector (stage d - 1, cyclically; its value is in registers since then)
                if (vd + (kDepth - 1) * kThreads < nv && GG_IN_BOUNDS(head + (int64_t)(vd + (kDepth - 1) * kThreads) * 8 + 7, n))
                    copy16<HINT>(slot0 + ((d + kDepth - 1) % kDepth) * kStageBytes, xv + (d + kDepth - 1) * kThreads,
                                 vd + (kDepth - 1) * kThreads < hints.split ? hints.first : hints.rest);
                asm volatile("cp.async.commit_group;" ::: "memory");
                asm volatile("cp.async.wait_group %0;" ::"n"(kDepth - 1) : "memory");
                uint4 r0;
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r0.x), "=r"(r0.y), "=r"(r0.z), "=r"(r0.w) : "r"(slot0 + d * kStageBytes) : "memory");
                TG *gd = gv != nullptr && GG_IN_BOUNDS(head + (int64_t)vd * 8 + 7, n) ? gv + (int64_t)d * kThreads * 8 : nullptr;
                process_vec<TG, FLAGS, MODE>(r0, gd, accumulate, wide, ln, sm, acc);
            }
        }
        xv += kDepth * kThreads;
        if (gv != nullptr) gv += kDepth * kThreads * 8;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// What a CTA carries from one run to the next: the key of the counts in shared memory and the lane constants.
struct CtaState {
    int cur_hid = -1, cur_mode = kModePattern;
    uint32_t cur_inv_bits = 0;
    bool have_key = false;
    Lane ln;
};

// Per-segment parameters: plain loads, or loads that bypass L1 when another CTA of the same launch wrote them.
template <bool COHERENT, typename T>
__device__ __forceinline__ T param(const T *p)
{
    if constexpr (COHERENT) return __ldcg(p);
    return *p;
}

__device__ __forceinline__ void init_cta(Smem &sm, CtaState &cs, bool hist)
{
    const int tid = threadIdx.x;
    if (hist) {
        for (int i = tid; i < (int)kCntWords; i += kThreads) sm.cnt[i] = 0u;
        for (int i = tid; i < kSymWin; i += kThreads) sm.win[i] = 0u;
        if (tid < 2) sm.clampc[tid] = 0u;
    }
    if (tid < 128) sm.lg[tid] = log2(1.0 + (double)tid * (1.0 / 128.0));
    if (tid == 0) { sm.cold.c_base = 0u; sm.cold.active = 0; sm.cold.sign_flip = 0u; sm.cold.symbol_mode = 0; }
    cs.ln.b_addr = (uint32_t)__cvta_generic_to_shared(sm.brep) + (uint32_t)(tid & 31) * 4u;
    // row r of the symbol table is reached as bits(floor(t) + magic) * 128 + s_addr (mod 2^32)
    cs.ln.s_addr = (uint32_t)__cvta_generic_to_shared(sm.cnt) + 128u + (uint32_t)(tid & 31) * 4u - kSymBase * 128u;
    cs.ln.p_addr = (uint32_t)__cvta_generic_to_shared(sm.cnt) + (uint32_t)(tid & (kRep - 1)) * 4u;
    cs.ln.cbase = 0x8000u;
    cs.ln.inv = 0.0f;
    cs.ln.inv2 = 0ull;
    __syncthreads();
}

// Gradient tables and count layout of the segment a run lies in; returns the count mode of the run.  x, n: the
// run (its first elements give the scale of the data when the caller does not know it).
template <int FLAGS, bool COHERENT>
__device__ __forceinline__ int setup_run(const StreamArgs &a, Smem &sm, CtaState &cs, int s, int64_t len, const uint16_t *x, int64_t n)
{
    constexpr bool GRAD = (FLAGS & kGrad) != 0, HIST = (FLAGS & kHist) != 0;
    const int tid = threadIdx.x;
    Lane &ln = cs.ln;
    int mode = kModePattern;
    bool active = false;

    if constexpr (GRAD && (FLAGS & kEg) != 0) {
        // code-length gradient: one factor per segment (Eq. 7 relaxed), no tables
        const float inv_s = (float)(1.0 / (double)param<COHERENT>(a.step + s));
        ln.eg_c = (float)(a.lambda * 4.0 * (double)inv_s / ((double)len * 0.6931471805599453094));
        ln.eg_two_k = 1u << a.eg_k;
        ln.qmin = a.qmin;
        ln.qmax = a.qmax;
        if (tid == 0) { sm.cold.active = 0; sm.cold.sign_flip = 0u; sm.cold.L = 0.0; sm.cold.b = 0.0; }
    } else if constexpr (GRAD) {
        const double beta = param<COHERENT>(a.beta + s), alpha = param<COHERENT>(a.alpha + s);
        const double lam = a.mean_reduction ? a.lambda / (double)len : a.lambda;
        active = (beta > 0.0) && (alpha > 0.0) && (lam != 0.0) && (lam == lam);
        // (every thread works the two constants out for itself: cheaper than a broadcast and its barrier)
        const double b = beta - 1.0;
        const double L = active ? log2(fabs(lam) * beta) - beta * log2(alpha) : 0.0;
        if (tid == 0) {
            sm.cold.b = b;
            sm.cold.sign_flip = lam < 0.0 ? 0x80000000u : 0u;
            sm.cold.active = active;
            sm.cold.L = L;
        }
        if (tid < 256) {
            const int k = tid;
            float2 v = make_float2(0.0f, 1.0f);
            if (active && k >= 1 && k <= 254) {
                const double e0 = L + b * (double)(k - 127);
                double ip = rint(e0);
                const double f = exp2_short(e0 - ip);
                ip = fmin(fmax(ip, -400.0), 400.0);
                const int ii = (int)ip;
                const int i1 = max(-100, min(100, ii));
                const int i2 = max(-126, min(126, ii - i1));
                v = make_float2((float)ldexp(lam < 0.0 ? -f : f, i1), __int_as_float((i2 + 127) << 23));
            }
            sm.A[k] = v;
            // One factor serves an exponent if its power-of-two part is 1 (|L + b (e-127)| <= 100:
            // the product with B then stays in the normal fp32 range).  Zero/subnormal (e = 0),
            // inf/nan (e = 255) and the far exponents get the marker.  Without a gradient all is zero.
            float one = 0.0f;
            if (active) one = (k >= 1 && k <= 254 && v.y == 1.0f) ? v.x : __int_as_float(0x7FC00000);
            s_a1[k] = one;
        } else if (tid < 384) {
            const int k = tid - 256;
            sm.B[k] = active ? (float)exp2_short(b * sm.lg[k]) : 1.0f;
        }
        __syncthreads();
        for (int i = tid; i < 128 * 32; i += kThreads) sm.brep[i] = sm.B[i >> 5];
    }
    if constexpr (HIST) {
        const int hid = a.map.hist_id ? a.map.hist_id[s] : s;
        const float step = param<COHERENT>(a.step + s);
        const float inv = (float)(1.0 / (double)step);
        const bool same_key = cs.have_key && hid == cs.cur_hid && __float_as_uint(inv) == cs.cur_inv_bits;
        // where the pattern-count window should sit: 16 binades below 2^5 standard deviations when
        // the scale of the data is known, else where it is (same key) or from four binades below
        // the step upwards (new key)
        uint32_t want_base = sm.cold.c_base;
        double sd = 0.0;
        if (a.seg_sd != nullptr) {
            sd = param<COHERENT>(a.seg_sd + s);
        } else {
            // Without parameters the scale of the data is taken from the first elements of the run (one
            // per thread): it only decides how the counts are laid out, never what is counted.
            const int m = (int)min(n, (int64_t)kThreads);
            float ss = 0.0f;
            for (int i = tid; i < m; i += kThreads) {
                const float v = __uint_as_float((uint32_t)__ldg(x + i) << 16);
                if (fabsf(v) <= 1e18f) ss = fmaf(v, v, ss);        // (inf, nan and values whose squares overflow are left out)
            }
            const double ws = warp_sum((double)ss);
            __syncthreads();                                        // (the slots may still be read from the run before)
            if ((tid & 31) == 0) sm.red[2][tid >> 5] = ws;
            __syncthreads();
            double tot = 0.0;
            for (int w = 0; w < kWarps; ++w) tot += sm.red[2][w];
            sd = m > 0 ? sqrt(tot / (double)m) : 0.0;
        }
        if (sd > 0.0) {
            want_base = (uint32_t)(window_top_exponent(sd, 4) - (kCntBinades - 1)) << 7;
            // symbol mode: the window's symbols are not clamped and reach 6.5 standard deviations
            if (a.qmin <= -(int)(kSymCells / 2) && a.qmax >= (int)(kSymCells / 2) - 1 && step > 0.0f &&
                (double)(kSymCells / 2) * (double)step >= 6.5 * sd && inv < 3.0e38f)
                mode = kModeSymbol;
        } else if (!same_key) {
            want_base = (uint32_t)(window_top_exponent((double)step, 11) - (kCntBinades - 1)) << 7;
        }
        const bool rebase = !same_key || mode != cs.cur_mode || (mode == kModePattern && want_base != sm.cold.c_base);
        __syncthreads();
        if (rebase) {
            if (cs.have_key) flush_counts(sm, a.clamped, cs.cur_hid);
            cs.have_key = true;
            cs.cur_hid = hid;
            cs.cur_inv_bits = __float_as_uint(inv);
            cs.cur_mode = mode;
            if (tid == 0) {
                sm.cold.inv = inv;
                sm.cold.qmin = a.qmin;
                sm.cold.qmax = a.qmax;
                sm.cold.row = reinterpret_cast<unsigned long long *>(a.hist) +
                              (int64_t)hid * ((int64_t)a.qmax - (int64_t)a.qmin + 1);
                sm.cold.c_base = want_base;
                sm.cold.symbol_mode = mode == kModeSymbol;
            }
        }
        ln.cbase = want_base;
        ln.inv = inv;
        ln.inv2 = pack2(inv, inv);
    }
    __syncthreads();
    return mode;
}

// The tiles [t_begin, t_end) of one CTA, run by run (a run: the tiles of the range that lie in one segment):
// gradient tables and count layout of the run's segment, then the stream, then the run's partial sums.
template <typename TG, int FLAGS, bool COHERENT, bool HINT>
__device__ __forceinline__ void tail_tiles(const StreamArgs &a, Smem &sm, CtaState &cs, int t_begin, int t_end, uint64_t policy)
{
    constexpr bool MOM = (FLAGS & kMoments) != 0, GRAD = (FLAGS & kGrad) != 0, HIST = (FLAGS & kHist) != 0;
    const bool accumulate = GRAD && a.accumulate != 0;
    Lane &ln = cs.ln;
    for (int t = t_begin; t < t_end;) {
        // ---- one run: the tiles of this CTA's range that lie in segment s
        const int s = a.map.tile_seg[t];
        const int64_t len = a.map.seg_len[s];
        const int t_first = a.map.tile_prefix[s];
        const int t_stop = min(t_end, a.map.tile_prefix[s + 1]);
        const int64_t off = (int64_t)(t - t_first) * kTile;
        const int64_t n = min(len, (int64_t)(t_stop - t_first) * kTile) - off;
        const uint16_t *x = reinterpret_cast<const uint16_t *>(a.map.seg_ptr[s]) + off;
        const int mode = setup_run<FLAGS, COHERENT>(a, sm, cs, s, len, x, n);

        // ---- stream the run
        TG *gout = nullptr;
        if constexpr (GRAD) {
            if (a.map.grad_ptr != nullptr) gout = reinterpret_cast<TG *>(a.map.grad_ptr[s]) + off;
        }
        Acc acc;
        Hints hints;
        hints.first = policy; hints.rest = policy; hints.split = 0;
        if constexpr (HIST) {
            if (mode == kModeSymbol) process_range<TG, FLAGS, kModeSymbol, HINT>(x, gout, n, accumulate, ln, sm, acc, hints);
            else process_range<TG, FLAGS, kModePattern, HINT>(x, gout, n, accumulate, ln, sm, acc, hints);
        } else {
            process_range<TG, FLAGS, kModePattern, HINT>(x, gout, n, accumulate, ln, sm, acc, hints);
        }

        if constexpr (MOM || GRAD) reduce_partials<FLAGS>(a.part, t, t_stop, acc, sm);
        else __syncthreads();
        t = t_stop;
    }
}

template <typename TG, int FLAGS>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) tail_bf16_kernel(const StreamArgs a)
{
    constexpr bool HIST = (FLAGS & kHist) != 0;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
    CtaState cs;
    init_cta(sm, cs, HIST);
    // contiguous range of tiles for this CTA
    const int64_t nt = a.map.n_tiles;
    const int t_begin = (int)(nt * blockIdx.x / gridDim.x);
    const int t_end = (int)(nt * (blockIdx.x + 1) / gridDim.x);
    tail_tiles<TG, FLAGS, false, false>(a, sm, cs, t_begin, t_end, 0);
    if constexpr (HIST) {
        if (cs.have_key) flush_counts(sm, a.clamped, cs.cur_hid);
    }
}

// ------------------------------------------------------------------------------------------------------------
// The whole fitted pass in ONE launch that keeps every tensor in L2 between its two reads.
//
// The segments are cut into groups of consecutive segments of about a quarter of L2 (one segment of any length
// is a group by itself).  All CTAs but the last are streamers and walk the groups together, each on its share
// of the group's tiles:
//     moments of group g            (the first `protect` part of the share is read with an evict-last hint)
//     arrive(g)
//     last tile of group g - 1      (gradient + counts; this tile was deferred to cover the wait below)
//     wait until the fit of group g is published
//     all but the last tile of group g   (gradient + counts; read again, now from L2, with an evict-first hint)
// The last CTA is the fitter: for every group it waits for all arrivals, adds the run partials of each of the
// group's segments in a fixed order, inverts the moment ratio and publishes the parameters.  The deferred tile
// is what hides the fitter's latency: without it every streamer would idle for a barrier and a fit per group.
// Every wait is bounded: when it runs out the CTA marks the segments GG_FLAG_TIMEOUT (fitter) and returns, and
// the others run out in turn.  The launch is cooperative, so all CTAs are resident and every wait can end.
__device__ __forceinline__ bool bounded_wait(const uint32_t *flag, uint32_t want, uint32_t cap, int *sh_ok)
{
    if (threadIdx.x == 0) {
        int ok = 0;
        for (uint32_t it = 0; it < cap; ++it) {
            uint32_t v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
            if (v >= want) { ok = 1; break; }
            __nanosleep(100);
        }
        __threadfence();
        *sh_ok = ok;
    }
    __syncthreads();
    const bool ok = *sh_ok != 0;
    __syncthreads();      // (the word is written again by the next wait)
    return ok;
}

__device__ __forceinline__ void publish(uint32_t *flag, bool add)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (add) atomicAdd(flag, 1u);
        else asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flag), "r"(1u) : "memory");
    }
}

__device__ __forceinline__ uint64_t make_policy(bool keep)
{
    uint64_t p;
    if (keep) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// Share of streamer b of the tiles [g0, g0 + n): [first, second).
__device__ __forceinline__ int2 share_of(int g0, int n, int b, int n_stream)
{
    return make_int2(g0 + (int)((int64_t)n * b / n_stream), g0 + (int)((int64_t)n * (b + 1) / n_stream));
}

__device__ void fitter(const StreamArgs &a, const ResidentArgs &r, int *sh_ok)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_stream = (int)gridDim.x - 1;
    for (int g = 0; g < r.n_groups; ++g) {
        if (!bounded_wait(r.arrive + g, r.expect, r.wait_cap, sh_ok)) {
            // nothing from here on can be trusted: say so per segment and stop (the streamers run out in turn)
            if (r.fit.flags != nullptr)
                for (int s = r.groups[g].z + tid; s < a.map.n_seg; s += kThreads) r.fit.flags[s] = GG_FLAG_TIMEOUT;
            return;
        }
        const int4 gr = r.groups[g];
        const int n = gr.y - gr.x;
        for (int s = gr.z + warp; s < gr.w; s += kWarps) {
            const int ts0 = a.map.tile_prefix[s], ts1 = a.map.tile_prefix[s + 1];
            double s1 = 0.0, s2 = 0.0;
            uint32_t bad = 0;
            float xmin = INFINITY, xmax = -INFINITY;
            // the runs of this segment: one per streamer whose share meets it, at the later of the two starts
            for (int b = lane; b < n_stream && ts1 > ts0; b += 32) {
                const int2 sh = share_of(gr.x, n, b, n_stream);
                const int t0 = max(sh.x, ts0);
                if (t0 >= min(sh.y, ts1)) continue;
                s1 += __ldcg(a.part.s1 + t0);
                s2 += __ldcg(a.part.s2 + t0);
                bad += __ldcg(a.part.bad + t0);
                xmin = fminf(xmin, __ldcg(a.part.xmin + t0));
                xmax = fmaxf(xmax, __ldcg(a.part.xmax + t0));
            }
            s1 = warp_sum(s1);
            s2 = warp_sum(s2);
            bad = __reduce_add_sync(0xFFFFFFFFu, bad);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                xmin = fminf(xmin, __shfl_xor_sync(0xFFFFFFFFu, xmin, o));
                xmax = fmaxf(xmax, __shfl_xor_sync(0xFFFFFFFFu, xmax, o));
            }
            fit_finish(r.fit, s, lane, s1, s2, bad, xmin, xmax);
        }
        publish(r.ready + g, false);
    }
}

template <typename TG, int FLAGS>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) resident_bf16_kernel(const StreamArgs a, const ResidentArgs r)
{
    constexpr bool HIST = (FLAGS & kHist) != 0;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
    __shared__ int sh_ok;
    const int n_stream = (int)gridDim.x - 1;
    if ((int)blockIdx.x == n_stream) { fitter(a, r, &sh_ok); return; }

    CtaState cs;
    init_cta(sm, cs, HIST);
    const uint64_t keep = make_policy(true), drop = make_policy(false);
    int late0 = 0, late1 = 0;      // the deferred last tile of the group before
    for (int g = 0; g < r.n_groups; ++g) {
        const int4 gr = r.groups[g];
        const int n = gr.y - gr.x;
        const int2 sh = share_of(gr.x, n, (int)blockIdx.x, n_stream);
        // ---- moments of this CTA's share, run by run
        // (of a group of more than keep_tiles tiles only the first keep_tiles / n of every share is asked to stay in L2)
        const int64_t share = sh.y - sh.x;
        const int t_keep = sh.x + (int)(n <= (int)r.keep_tiles ? share : (share * r.keep_tiles + n - 1) / n);
        for (int t = sh.x; t < sh.y;) {
            const int s = a.map.tile_seg[t];
            const int64_t len = a.map.seg_len[s];
            const int t_first = a.map.tile_prefix[s];
            const int t_stop = min(sh.y, a.map.tile_prefix[s + 1]);
            const int64_t off = (int64_t)(t - t_first) * kTile;
            const int64_t n_el = min(len, (int64_t)(t_stop - t_first) * kTile) - off;
            const uint16_t *x = reinterpret_cast<const uint16_t *>(a.map.seg_ptr[s]) + off;
            Hints hints;
            hints.first = keep; hints.rest = drop;
            hints.split = (int)min((int64_t)max(t_keep - t, 0) * (kTile / 8), (int64_t)0x7FFFFFFF);
            Acc acc;
            process_range<float, kMoments, kModePattern, true>(x, nullptr, n_el, false, cs.ln, sm, acc, hints);
            reduce_partials<kMoments>(a.part, t, t_stop, acc, sm);
            t = t_stop;
        }
        publish(r.arrive + g, true);
        if (late1 > late0) tail_tiles<TG, FLAGS, true, true>(a, sm, cs, late0, late1, drop);
        if (!bounded_wait(r.ready + g, 1u, 2u * r.wait_cap, &sh_ok)) return;
        late0 = sh.y - sh.x >= 2 ? sh.y - 1 : sh.y;
        late1 = sh.y;
        tail_tiles<TG, FLAGS, true, true>(a, sm, cs, sh.x, late0, drop);
    }
    if (late1 > late0) tail_tiles<TG, FLAGS, true, true>(a, sm, cs, late0, late1, drop);
    if constexpr (HIST) {
        if (cs.have_key) flush_counts(sm, a.clamped, cs.cur_hid);
    }
}

// ------------------------------------------------------------------------------------------------------------
// The fitted pass for segments of tens of kilobytes to two megabytes with ONE read of x from DRAM: a thread-block
// cluster per segment, the segment staged in the shared memory of the cluster's CTAs.
//
// CTA r of a cluster of C takes the r-th share of the segment's tiles (at most kClusterTiles tiles) and copies it
// into its shared memory with bulk asynchronous copies that complete on an mbarrier.  Moments come from shared
// memory; every CTA leaves its sums in a slot of its own shared memory, the cluster synchronises (the hardware
// barrier of the cluster: its CTAs are scheduled together), and the first warp of every CTA adds the C slots in
// rank order through distributed shared memory and inverts the moment ratio: every CTA ends with the same bits and
// nothing else is exchanged.  Gradient tables, gradient, penalty partial and counts then come from the staged copy.
// Clusters are independent of one another, so while one waits for its barrier or works on a fit the others keep
// DRAM busy.  The wait for the bulk copies is bounded; if it runs out the CTA stops touching data, keeps taking part
// in the cluster barriers and marks its segments GG_FLAG_TIMEOUT at the end.
constexpr int kClusterTiles = 4;                                     // tiles of a segment one CTA can stage (128 KB)
constexpr size_t kClusterSmem = sizeof(Smem) - sizeof(uint4) * kDepth * kThreads + (size_t)kClusterTiles * kTile * 2;

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t cap)
{
    for (uint32_t it = 0; it < cap; ++it) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

template <typename TG, int FLAGS>
__global__ void __launch_bounds__(kThreads, 1) cluster_bf16_kernel(const StreamArgs a, const ClusterArgs c)
{
    namespace cg = cooperative_groups;
    constexpr bool GRAD = (FLAGS & kGrad) != 0, HIST = (FLAGS & kHist) != 0;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
    const int cid = (int)blockIdx.x / C, n_clusters = (int)gridDim.x / C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    CtaState cs;
    init_cta(sm, cs, HIST);
    const uint4 *data = &sm.stage[0][0];
    const uint32_t data_addr = (uint32_t)__cvta_generic_to_shared(data), bar = (uint32_t)__cvta_generic_to_shared(&sm.mbar);
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool accumulate = GRAD && a.accumulate != 0;
    uint32_t parity = 0;
    int s_fail = -1;                // first segment whose copies did not arrive in time
    uint32_t fail_parity = 0;
    int it = 0;
    for (int s = cid; s < a.map.n_seg; s += n_clusters, ++it) {
        // ---- this CTA's share of the segment
        const int64_t len = a.map.seg_len[s];
        const int t0 = a.map.tile_prefix[s], T = a.map.tile_prefix[s + 1] - t0;
        const int t_lo = t0 + (int)((int64_t)T * rank / C), t_hi = t0 + (int)((int64_t)T * (rank + 1) / C);
        const int64_t off = (int64_t)(t_lo - t0) * kTile;
        const int n = t_hi > t_lo && s_fail < 0 ? (int)(min(len, (int64_t)(t_hi - t0) * kTile) - off) : 0;
        const uint16_t *x = reinterpret_cast<const uint16_t *>(a.map.seg_ptr[s]) + off;
        const int nvec = n / 8;

        // ---- stage it: bulk copies of up to one tile each, all completing on the one barrier
        bool ok = true;
        if (nvec > 0) {
            if (tid == 0 && GG_IN_BOUNDS(off + (int64_t)nvec * 8 - 1, len) && GG_IN_BOUNDS(nvec - 1, kClusterTiles * kTile / 8)) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the reads of the segment before are done
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)nvec * 16u + c.extra_tx) : "memory");
                for (int v0 = 0; v0 < nvec; v0 += kTile / 8) {
                    const uint32_t bytes = (uint32_t)min(nvec - v0, kTile / 8) * 16u;
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                                     data_addr + (uint32_t)v0 * 16u),
                                 "l"(reinterpret_cast<const uint4 *>(x) + v0), "r"(bytes), "r"(bar)
                                 : "memory");
                }
            }
            ok = mbar_wait(bar, parity, c.wait_cap);
            if (!ok) ok = mbar_wait(bar, parity, c.wait_cap);      // once more before giving up
            if (ok) parity ^= 1u;
        }
        if (__syncthreads_or(!ok)) {
            // (no further copy is issued by this CTA; the one in flight is waited for again before the CTA leaves)
            if (s_fail < 0) { s_fail = s; fail_parity = parity; }
            ok = false;
        }

        // ---- moments of the share, from shared memory
        Acc acc;
        if (ok) {
            for (int v = tid; v < nvec; v += kThreads) process_vec<float, kMoments, kModePattern>(data[v], nullptr, false, false, cs.ln, sm, acc);
            for (int i = nvec * 8 + tid; i < n; i += kThreads) scalar_elem<float, kMoments, kModePattern>(x, nullptr, i, false, cs.ln, sm, acc);
        }
        {
            const double w1 = warp_sum(acc.s1), w2 = warp_sum(acc.s2);
            const uint32_t wb = __reduce_add_sync(0xFFFFFFFFu, acc.bad);
            float wmin = fminf(acc.xmin, fminf(__low2float(acc.mn2), __high2float(acc.mn2)));
            float wmax = fmaxf(acc.xmax, fmaxf(__low2float(acc.mx2), __high2float(acc.mx2)));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                wmin = fminf(wmin, __shfl_xor_sync(0xFFFFFFFFu, wmin, o));
                wmax = fmaxf(wmax, __shfl_xor_sync(0xFFFFFFFFu, wmax, o));
            }
            if (lane == 0) { sm.red[0][warp] = w1; sm.red[1][warp] = w2; sm.bad[warp] = wb; sm.mn[warp] = wmin; sm.mx[warp] = wmax; }
            __syncthreads();
            if (tid == 0) {
                ClusterPart p{0.0, 0.0, 0u, INFINITY, -INFINITY};
                for (int w = 0; w < kWarps; ++w) {
                    p.s1 += sm.red[0][w]; p.s2 += sm.red[1][w]; p.bad += sm.bad[w];
                    p.mn = fminf(p.mn, sm.mn[w]); p.mx = fmaxf(p.mx, sm.mx[w]);
                }
                sm.cpart[it & 1] = p;
            }
        }
        cluster.sync();

        // ---- the fit, by the first warp of every CTA: the C slots in rank order, the same bits everywhere
        if (warp == 0) {
            double s1 = 0.0, s2 = 0.0;
            uint32_t bad = 0;
            float xmin = INFINITY, xmax = -INFINITY;
            for (int r = 0; r < C; ++r) {
                const ClusterPart *p = cluster.map_shared_rank(&sm.cpart[it & 1], r);
                s1 += p->s1; s2 += p->s2; bad += p->bad;
                xmin = fminf(xmin, p->mn); xmax = fmaxf(xmax, p->mx);
            }
            fit_finish(c.fit, s, lane, s1, s2, bad, xmin, xmax);      // (every CTA writes the same values to the outputs)
        }
        __syncthreads();

        // ---- gradient tables, then gradient, penalty partial and counts from the staged copy
        if (ok && n > 0) {
            const int mode = setup_run<FLAGS, false>(a, sm, cs, s, len, x, n);
            TG *gout = nullptr;
            if constexpr (GRAD) {
                if (a.map.grad_ptr != nullptr) gout = reinterpret_cast<TG *>(a.map.grad_ptr[s]) + off;
            }
            TG *gv = gout != nullptr ? gout + (int64_t)tid * 8 : nullptr;
            const bool wide = (reinterpret_cast<uintptr_t>(gv) & 31u) == 0;
            Acc acc2;
            auto second = [&](auto mode_tag) {
                constexpr int MODE = decltype(mode_tag)::value;
                for (int v = tid; v < nvec; v += kThreads)
                    process_vec<TG, FLAGS, MODE>(data[v], gout != nullptr ? gout + (int64_t)v * 8 : nullptr, accumulate, wide, cs.ln, sm, acc2);
                for (int i = nvec * 8 + tid; i < n; i += kThreads) scalar_elem<TG, FLAGS, MODE>(x, gout, i, accumulate, cs.ln, sm, acc2);
            };
            if (HIST && mode == kModeSymbol) second(std::integral_constant<int, kModeSymbol>());
            else second(std::integral_constant<int, kModePattern>());
            if constexpr (GRAD) reduce_partials<FLAGS>(a.part, t_lo, t_hi, acc2, sm);
            else __syncthreads();
        } else if (GRAD && t_hi > t_lo) {
            for (int t = t_lo + tid; t < t_hi; t += kThreads) a.part.pen[t] = 0.0;
        }
    }
    if constexpr (HIST) {
        if (cs.have_key) flush_counts(sm, a.clamped, cs.cur_hid);
    }
    cluster.sync();       // nobody leaves while another CTA may still read its slots
    if (s_fail >= 0) {
        // (the copies that were late must not land in memory this CTA has given up)
        mbar_wait(bar, fail_parity, c.wait_cap < (1u << 16) ? c.wait_cap * 64u : (1u << 22));
        if (c.fit.flags != nullptr && tid == 0)
            for (int s = s_fail; s < a.map.n_seg; s += n_clusters) atomicOr(c.fit.flags + s, GG_FLAG_TIMEOUT);
    }
}

template <typename TG, int FLAGS>
cudaError_t launch_one(const StreamArgs &a, int sm_count, cudaStream_t st)
{
    auto kern = tail_bf16_kernel<TG, FLAGS>;
    // more than 48 KB of dynamic shared memory needs the opt-in (per function and device)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem));
    if (e != cudaSuccess) return e;
    const int grid = (int)min((int64_t)a.map.n_tiles, (int64_t)sm_count * kCtasPerSm);
    kern<<<grid, kThreads, sizeof(Smem), st>>>(a);
    return cudaGetLastError();
}

template <typename TG>
cudaError_t launch_typed(int flags, const StreamArgs &a, int sm_count, cudaStream_t st)
{
    switch (flags) {
    case kGrad: return launch_one<TG, kGrad>(a, sm_count, st);
    case kHist: return launch_one<TG, kHist>(a, sm_count, st);
    case kGrad | kHist: return launch_one<TG, kGrad | kHist>(a, sm_count, st);
    case kMoments | kGrad: return launch_one<TG, kMoments | kGrad>(a, sm_count, st);
    case kMoments | kHist: return launch_one<TG, kMoments | kHist>(a, sm_count, st);
    case kMoments | kGrad | kHist: return launch_one<TG, kMoments | kGrad | kHist>(a, sm_count, st);
    case kMoments | kGrad | kHist | kEg: return launch_one<TG, kMoments | kGrad | kHist | kEg>(a, sm_count, st);
    default: return cudaErrorInvalidValue;
    }
}

template <typename TG, int FLAGS>
cudaError_t resident_one(const StreamArgs &a, const ResidentArgs &r, int grid, int *max_grid, cudaStream_t st)
{
    auto kern = resident_bf16_kernel<TG, FLAGS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem));
    if (e != cudaSuccess) return e;
    if (max_grid != nullptr) {
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, sizeof(Smem));
        if (e != cudaSuccess) return e;
        *max_grid = per_sm * grid;      // (grid: the number of SMs)
        return cudaSuccess;
    }
    void *args[] = {const_cast<StreamArgs *>(&a), const_cast<ResidentArgs *>(&r)};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(kern), dim3((unsigned)grid), dim3(kThreads), args,
                                       sizeof(Smem), st);
}

template <typename TG>
cudaError_t resident_typed(int flags, const StreamArgs &a, const ResidentArgs &r, int grid, int *max_grid, cudaStream_t st)
{
    switch (flags) {
    case kGrad: return resident_one<TG, kGrad>(a, r, grid, max_grid, st);
    case kHist: return resident_one<TG, kHist>(a, r, grid, max_grid, st);
    case kGrad | kHist: return resident_one<TG, kGrad | kHist>(a, r, grid, max_grid, st);
    default: return cudaErrorInvalidValue;
    }
}

template <typename TG, int FLAGS>
cudaError_t cluster_one(const StreamArgs &a, const ClusterArgs &c, int cluster_size, int n_clusters, int *max_clusters, cudaStream_t st)
{
    auto kern = cluster_bf16_kernel<TG, FLAGS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kClusterSmem);
    if (e != cudaSuccess) return e;
    if (cluster_size > 8) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cluster_size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kClusterSmem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (max_clusters != nullptr) {
        cfg.gridDim = dim3((unsigned)cluster_size);
        return cudaOccupancyMaxActiveClusters(max_clusters, kern, &cfg);
    }
    cfg.gridDim = dim3((unsigned)(cluster_size * n_clusters));
    return cudaLaunchKernelEx(&cfg, kern, a, c);
}

template <typename TG>
cudaError_t cluster_typed(int flags, const StreamArgs &a, const ClusterArgs &c, int cluster_size, int n_clusters, int *max_clusters,
                          cudaStream_t st)
{
    switch (flags) {
    case kGrad: return cluster_one<TG, kGrad>(a, c, cluster_size, n_clusters, max_clusters, st);
    case kHist: return cluster_one<TG, kHist>(a, c, cluster_size, n_clusters, max_clusters, st);
    case kGrad | kHist: return cluster_one<TG, kGrad | kHist>(a, c, cluster_size, n_clusters, max_clusters, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_tail_bf16(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a,
                             int sm_count, cudaStream_t st)
{
    if (a.map.n_tiles <= 0) return cudaSuccess;
    if (has_grad_out && grad_dtype == GG_BF16) return launch_typed<uint16_t>(flags, a, sm_count, st);
    return launch_typed<float>(flags, a, sm_count, st);
}

cudaError_t launch_resident_bf16(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a,
                                 const ResidentArgs &r, int grid, cudaStream_t st)
{
    if (r.n_groups <= 0) return cudaSuccess;
    if (has_grad_out && grad_dtype == GG_BF16) return resident_typed<uint16_t>(flags, a, r, grid, nullptr, st);
    return resident_typed<float>(flags, a, r, grid, nullptr, st);
}

cudaError_t resident_bf16_max_grid(int flags, gg_dtype grad_dtype, bool has_grad_out, int sm_count, int *max_grid)
{
    StreamArgs a{};
    ResidentArgs r{};
    if (has_grad_out && grad_dtype == GG_BF16) return resident_typed<uint16_t>(flags, a, r, sm_count, max_grid, nullptr);
    return resident_typed<float>(flags, a, r, sm_count, max_grid, nullptr);
}

cudaError_t launch_cluster_bf16(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a, const ClusterArgs &c,
                                int cluster_size, int n_clusters, cudaStream_t st)
{
    if (n_clusters <= 0) return cudaSuccess;
    if (has_grad_out && grad_dtype == GG_BF16) return cluster_typed<uint16_t>(flags, a, c, cluster_size, n_clusters, nullptr, st);
    return cluster_typed<float>(flags, a, c, cluster_size, n_clusters, nullptr, st);
}

cudaError_t cluster_bf16_max_clusters(int flags, gg_dtype grad_dtype, bool has_grad_out, int cluster_size, int *max_clusters)
{
    StreamArgs a{};
    ClusterArgs c{};
    if (has_grad_out && grad_dtype == GG_BF16) return cluster_typed<uint16_t>(flags, a, c, cluster_size, 0, max_clusters, nullptr);
    return cluster_typed<float>(flags, a, c, cluster_size, 0, max_clusters, nullptr);
}

int cluster_tiles_per_cta() { return kClusterTiles; }

}  // namespace gg
