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

// One thread per count cell walks the CTA slots in order and adds up the runs of slots that share a
// key (histogram, step, window); each run becomes one symbol and one 64-bit addition.  With one key
// for the whole call, the usual case, that is one addition per cell.
// SYMBOLS false: the cells are bf16 bit patterns (kCells of them, key after them); true: the cells are symbols
// -kSymWin/2 .. kSymWin/2 - 1 between two sentinel cells (kSymWin + 2 of them, key after them).
constexpr uint32_t kSymWin = 8192;
template <bool SYMBOLS>
static __global__ void flush_slots_kernel(const uint32_t *__restrict__ cta_counts, int n_slots, int32_t qmin, int32_t qmax, uint64_t *hist,
                                   uint64_t *clamped)
{
    // the slots' keys first, into shared memory: scanning them from global memory would be one
    // dependent cache miss per slot
    __shared__ uint32_t sh_key[kMaxSlots][4];
    for (int b = threadIdx.y * blockDim.x + threadIdx.x; b < n_slots; b += blockDim.x * blockDim.y) {
        const uint32_t *key = cta_counts + (size_t)b * kSmallSlotWords + (SYMBOLS ? kSymWin + 2 : kCells);
#pragma unroll
        for (int q = 0; q < 4; ++q) sh_key[b][q] = __ldg(key + q);
    }
    __syncthreads();
    // thread (x, y): cell blockIdx.x * blockDim.x + x, the y-th of blockDim.y contiguous parts of the slots
    // (additions commute, so every part may emit its own runs)
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    if constexpr (SYMBOLS) {
        if (c == 0 || c > kSymWin) return;                                // (the two sentinel cells are not counted)
    } else {
        if (c >= kCells || c == kSentinel || c == kSentinel + 1) return;     // (the sentinel pair is not counted)
    }
    const int per_part = (n_slots + (int)blockDim.y - 1) / (int)blockDim.y;
    const int b_first = (int)threadIdx.y * per_part, b_last = min(n_slots, b_first + per_part);
    const int64_t n_bins = (int64_t)qmax - (int64_t)qmin + 1;
    unsigned long long run = 0;
    uint32_t k_hid = 0, k_inv = 0, k_base = 0;
    auto emit = [&]() {
        if (run == 0) return;
        int q;
        if constexpr (SYMBOLS) {
            q = (int)c - 1 - (int)(kSymWin / 2);
        } else if (c < kSentinel) {
            const uint32_t h = (k_base + (c >> 1)) | ((c & 1u) << 15);
            q = __float2int_rd(__fmul_rn(__uint_as_float(h << 16), __uint_as_float(k_inv)));   // (window patterns are finite)
        } else {
            q = c == kBelow ? 0 : -1;           // the values below the window
        }
        unsigned long long *cl = reinterpret_cast<unsigned long long *>(clamped);
        if (q < qmin) { q = qmin; if (cl) atomicAdd(cl + 2 * k_hid, run); }
        else if (q > qmax) { q = qmax; if (cl) atomicAdd(cl + 2 * k_hid + 1, run); }
        atomicAdd(reinterpret_cast<unsigned long long *>(hist) + (int64_t)k_hid * n_bins + (q - qmin), run);
        run = 0;
    };
    // (the keys are the same words for every thread: cached; the sums over a run are independent
    // loads, unrolled so that many are in flight)
    int b = b_first;
    while (b < b_last) {
        if (sh_key[b][0] == 0u) { ++b; continue; }                        // this CTA had no table (its cells are zeros)
        k_hid = sh_key[b][1]; k_inv = sh_key[b][2]; k_base = sh_key[b][3];
        int e = b + 1;
        for (; e < b_last; ++e) {
            if (sh_key[e][0] != 0u && (sh_key[e][1] != k_hid || sh_key[e][2] != k_inv || (!SYMBOLS && sh_key[e][3] != k_base))) break;
        }
        int i = b;
        for (; i + 16 <= e; i += 16) {
            uint32_t t[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) t[u] = __ldg(cta_counts + (size_t)(i + u) * kSmallSlotWords + c);
#pragma unroll
            for (int u = 0; u < 16; ++u) run += t[u];
        }
        for (; i < e; ++i) run += __ldg(cta_counts + (size_t)i * kSmallSlotWords + c);
        emit();
        b = e;
    }
}


}  // namespace gg
