// Pieces shared by the kernels that run the whole pass for short segments (one warp or one team of warps per
// segment): the CTA-wide pattern-count table of bf16 input and the cold paths.
#pragma once
#include <stdint.h>

#include "gg_internal.h"

namespace gg {

constexpr int kCntBinades = 32;
constexpr uint32_t kCntPat = kCntBinades * 128;
// count cells of a CTA: two per pattern of the window (sign), the sentinel pair that swallows the
// first-pass counts of values outside the window, and the pair for values below the window
constexpr uint32_t kSentinel = kCntPat * 2, kBelow = kCntPat * 2 + 2;
constexpr uint32_t kCells = kCntPat * 2 + 4;
static_assert(kCells + 4 <= (uint32_t)kSmallSlotWords, "scratch slot");
constexpr int kMaxSlots = 1024;      // CTAs of one launch whose tables the flush kernel can take


// The gradient magnitude in fp64 for one magnitude pattern: the exact path.  The caller adds its
// penalty term |x| |g| before rounding the gradient to fp32 (which may underflow or overflow).
static __device__ __noinline__ double grad_fp64(uint32_t mag, double L, double b, bool active)
{
    const float ax = __uint_as_float(mag << 16);
    if (!active || ax == 0.0f) return 0.0;
    return exp2(L + b * log2((double)ax));
}

// Quantises one value and counts its symbol in global memory (elements the CTA table does not serve).
// Returns 1 / 2 if the symbol was clamped at the low / high end, else 0.  (Everything by value: a
// structure passed by reference to a function that is not inlined would live in local memory.)
static __device__ __noinline__ int count_global(uint32_t xb, float inv, int32_t qmin, int32_t qmax, unsigned long long *row)
{
    const float t = __fmul_rn(__uint_as_float(xb), inv);
    int clamped = 0;
    if (t == t) {                               // NaN is skipped
        int q = __float2int_rd(t);              // floor, saturating
        if (q < qmin) { q = qmin; clamped = 1; }
        else if (q > qmax) { q = qmax; clamped = 2; }
        atomicAdd(&row[q - qmin], 1ull);
    }
    return clamped;
}

// Exponent field of the top binade of the CTA's pattern-count window: 2^11 steps.
static __device__ __forceinline__ int window_top_exponent(double step)
{
    int e = 127 + 11;
    if (step > 0.0 && step < 1e300) e = ilogb(step) + 127 + 11;
    return max(kCntBinades, min(254, e));
}

}  // namespace gg
