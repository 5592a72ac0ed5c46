// fp32-input sweep with a gradient and/or a histogram (and, when the parameters are given, the moments of the
// next fit in the same read): the counterpart of the bf16 pattern kernel for tensors whose elements are full
// fp32 numbers (gradient buckets and the like).
//
// Persistent CTAs each walk one contiguous range of tiles; inside a segment that is one contiguous
// run of elements, streamed as pairs of 128-bit vectors through a per-thread ring of shared-memory
// slots filled by asynchronous copies (bytes in flight cost no registers).
//   * gradient: |x| = 2^e m with m in [1, 2); c = 1 + j/128 is m cut to its top 7 fraction bits, so
//     d = m - c is exact and r = d / c < 2^-7.  Then
//         |g| = A[e] * B[j] * (1 + r)^b,   A[e] = 2^(L + b (e-127)),   B[j] = c^b,
//     with A indexed by the exponent field, B replicated once per shared-memory bank, 1/c from the
//     reciprocal unit (its error enters multiplied by b r: below 2^-29) and (1 + r)^b as the
//     degree-4 binomial series (next term below 2e-10 for |b| <= 2).  Roundings: A, B, the fused
//     B + B t, and the product: within 2.5 ulp.  Exponents that A cannot serve as one normal fp32
//     factor (zero/subnormal, inf/nan, far binades), and every exponent when |b| > 2, hold NaN;
//     the NaN reaches the penalty partial of the vector, whose range check sends the vector to the
//     fp64 path.
//   * histogram: by quantised symbol, floor(x * inv) taken with a round-down add of 1.5 * 2^23 after
//     clamping x * inv to just outside the count window.  Two layouts of the window: rows of 32
//     words per symbol with lane l counting in word l when 128 steps reach 6.5 standard deviations
//     (the atomic is then free of bank conflicts), else one word per symbol over [-4096, 4096).
//     A symbol outside the window lands on a sentinel and is counted again in global memory.
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
constexpr int kDepth = 3;                           // pairs of input vectors staged ahead per thread
constexpr uint32_t kSymCells = 256;                 // row layout: symbols [-128, 128)
constexpr uint32_t kWinCells = 8192;                // word layout: symbols [-4096, 4096)
constexpr uint32_t kCntWords = (kSymCells + 2) * 32 > kWinCells + 2 ? (kSymCells + 2) * 32 : kWinCells + 2;
enum : int { kModeWords = 1, kModeRows = 2 };

// Constants of the current segment / histogram that only the cold paths need.
struct Cold {
    double L, b;               // g = 2^(L + b log2|x|)
    uint32_t sign_flip;        // 0x80000000 if lambda < 0 (the tables then hold -|g|)
    int active;                // 0: the gradient is zero everywhere
    float inv;                 // quantiser: q = floor(x * inv)
    int32_t qmin, qmax;
    unsigned long long *row;   // the current histogram, bin 0 = symbol qmin
    int rows_mode;             // layout of cnt: 1 = rows of 32 words per symbol, 0 = one word per symbol
};

struct Smem {
    // rows: word ((s + 1) * 32 + lane) = symbol s - kSymCells/2 counted by that lane; words: word
    // (s + 1) = symbol s - kWinCells/2.  Row / word 0 and the last one are the sentinels of the tails.
    uint32_t cnt[kCntWords];
    uint4 stage[kDepth][2][kThreads];   // per-thread ring: two 16-byte vectors (eight elements) per slot
    float brep[128 * 32];               // row j: B[j] = (1 + j/128)^b in every bank
    float B[128];
    double lg[128];                     // log2(1 + j/128)
    double red[3][kWarps];             // sum |x|, sum x^2, sum |x| |g| of the warps
    uint32_t bad[kWarps];
    float mn[kWarps], mx[kWarps];
    uint32_t clampc[2];
    Cold cold;
};

// Per-thread sums of one run.
struct Acc {
    double s1 = 0.0, s2 = 0.0, pen = 0.0;
    uint32_t bad = 0;
    float xmin = INFINITY, xmax = -INFINITY;
};

// A[e] as one factor (with lambda's sign), NaN where that is not possible.  Static shared memory:
// its address is a compile-time constant, so a look-up is an index and a load.
__shared__ float s_a1[256];

// |g| (with lambda's sign) in fp64 for any input: the exact path.
__device__ __noinline__ float grad_exact(uint32_t xb, double L, double b, int active, uint32_t sign_flip)
{
    const float ax = __uint_as_float(xb & 0x7FFFFFFFu);
    if (!active || ax == 0.0f) return 0.0f;
    const float v = (float)exp2(L + b * log2((double)ax));     // round to nearest: overflow -> inf, subnormals rounded once
    return __uint_as_float(__float_as_uint(v) ^ sign_flip);
}

// Quantises one value and counts its symbol in global memory (symbols the window does not hold).
// Returns 1 / 2 if the symbol was clamped at the low / high end, else 0.
__device__ __noinline__ int count_global(uint32_t xb, float inv, int32_t qmin, int32_t qmax, unsigned long long *row)
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

// Per-thread constants of the element path.
struct Lane {
    uint32_t b_addr;   // shared address of brep + lane * 4
    uint32_t c_addr;   // count address base: see one_elem
    float inv;         // quantiser scale
    float c1, c2, c3, c4;   // binomial coefficients of (1 + r)^b
    float eg_c;        // code-length gradient (kEg): the factor c of the segment, 2^k, the clamp of the symbols
    uint32_t eg_two_k;
    int32_t qmin, qmax;
};

template <int MODE> struct Window;
template <> struct Window<kModeRows> {
    static constexpr float kHalf = (float)(kSymCells / 2);
    static constexpr uint32_t kShift = 7;      // 128 bytes per symbol
};
template <> struct Window<kModeWords> {
    static constexpr float kHalf = (float)(kWinCells / 2);
    static constexpr uint32_t kShift = 2;      // 4 bytes per symbol
};

// One element (fp32 bits).  Branch free.  Gradient: a NaN entry of s_a1 makes the vector's penalty
// partial NaN, which the caller checks once per vector.  Count: `anyt` keeps the largest |x * inv|
// so that one compare per vector finds symbols outside the window; those count on a sentinel.
template <int FLAGS, int MODE>
__device__ __forceinline__ float one_elem(uint32_t xb, const Lane &ln, float &mp, float &anyt, float &m1, float &m2, Acc &acc)
{
    float ga = 0.0f;
    const float x = __uint_as_float(xb);
    if constexpr ((FLAGS & kMoments) != 0) {
        // fp32 sums of the vector; an inf or nan makes them inf or nan, and the vector is then summed again in fp64
        m1 += fabsf(x);
        m2 = fmaf(x, x, m2);
        acc.xmin = fminf(acc.xmin, x);          // fminf / fmaxf return the non-NaN operand
        acc.xmax = fmaxf(acc.xmax, x);
    }
    constexpr bool EG = (FLAGS & kEg) != 0;
    if constexpr ((FLAGS & kGrad) != 0 && !EG) {
        const uint32_t ax = xb & 0x7FFFFFFFu;
        const float a = *reinterpret_cast<const float *>(reinterpret_cast<const char *>(s_a1) + ((ax >> 21) & 0x3FCu));
        const float bj = lds_f32(((ax >> 16) & 127u) * 128u + ln.b_addr);
        const float c = __uint_as_float((ax & 0x007F0000u) | 0x3F800000u);      // 1 + j/128
        const float m = __uint_as_float((ax & 0x007FFFFFu) | 0x3F800000u);
        const float r = (m - c) * rcp_approx(c);                                 // m = c (1 + r), m - c exact
        const float t = r * fmaf(r, fmaf(r, fmaf(r, ln.c4, ln.c3), ln.c2), ln.c1);   // (1 + r)^b - 1
        ga = a * fmaf(bj, t, bj);
        mp = fmaf(fabsf(x), fabsf(ga), mp);
    }
    if constexpr ((FLAGS & kHist) != 0) {
        const float t = __fmul_rn(x, ln.inv);
        // (a nan leaves anyt alone, see count_miss; with the code-length gradient it must be found, since its gradient
        // is zero and not the sentinel's: the maximum is then taken on the bit patterns, where a nan is the largest)
        if constexpr (EG) anyt = __uint_as_float(max(__float_as_uint(anyt), __float_as_uint(fabsf(t))));
        else anyt = fmaxf(anyt, fabsf(t));
        // t clamped to just outside the window: the floor of the clamped value lands on a sentinel for
        // either tail (and for nan, which the maximum replaces by the lower bound)
        const float tc = fminf(fmaxf(t, -Window<MODE>::kHalf - 0.5f), Window<MODE>::kHalf);
        // for |t| < 2^22 the sum lies in [2^23, 2^24) where floats are the integers: rounding down gives floor
        const uint32_t fb = __float_as_uint(__fadd_rd(tc, __uint_as_float(kMagicBits)));
        red_inc((fb << Window<MODE>::kShift) + ln.c_addr);   // (c_addr holds minus the shifted bits of the first symbol)
        if constexpr (EG) {
            // the symbol of an element inside the window (one outside is redone by fix_elem); zero has no gradient
            const int q = max(ln.qmin, min(ln.qmax, (int)(fb - kMagicBits)));
            ga = (xb << 1) != 0u ? eg_grad_of_symbol(q, ln.eg_c, ln.eg_two_k) : 0.0f;
        }
    }
    if constexpr ((FLAGS & kGrad) != 0)
        return __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));   // the table carries lambda's sign
    return 0.0f;
}

// Some |x * inv| reached the edge of the window.  (A nan input is not seen here: it counts on a
// sentinel and, being skipped by the quantiser, needs no second count.  With a gradient it is
// found through the penalty partial.)
template <int MODE>
__device__ __forceinline__ bool count_miss(float anyt) { return !(anyt < Window<MODE>::kHalf); }      // (a nan counts as a miss)

// Redo of whatever part of an element the branch-free path could not do; g is the gradient from the
// first pass.  grad_bad: the vector's penalty partial left the fp32 range.
template <int FLAGS, int MODE>
__device__ __forceinline__ float fix_elem(uint32_t xb, float g, bool grad_bad, const Lane &ln, Smem &sm, uint32_t (&clampc)[2])
{
    if constexpr ((FLAGS & kGrad) != 0 && (FLAGS & kEg) == 0) {
        if (grad_bad) {
            const float a = s_a1[(xb >> 23) & 0xFFu];
            if (a != a) {     // this element read a NaN marker
                const float ga = grad_exact(xb, sm.cold.L, sm.cold.b, sm.cold.active, sm.cold.sign_flip);
                g = __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));
            }
        }
    }
    if constexpr ((FLAGS & kHist) != 0) {
        const float t = __fmul_rn(__uint_as_float(xb), ln.inv);
        // outside the window (the exact test: floor(t) not in [-half, half))
        if (t >= Window<MODE>::kHalf || t < -Window<MODE>::kHalf) {
            const int c = count_global(xb, ln.inv, sm.cold.qmin, sm.cold.qmax, sm.cold.row);
            if (c) clampc[c - 1] += 1u;
        }
        if constexpr ((FLAGS & kEg) != 0) {
            if (!(t < Window<MODE>::kHalf && t >= -Window<MODE>::kHalf)) g = eg_grad_exact(xb, ln.inv, ln.qmin, ln.qmax, ln.eg_c, ln.eg_two_k);
        }
    }
    return g;
}

// fp64 penalty terms |x| |g| of eight values (a vector whose fp32 partial left the range).
__device__ __noinline__ double pen_exact(uint4 lo, uint4 hi, int n, double L, double b, int active)
{
    if (!active) return 0.0;
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    double dp = 0.0;
    for (int e = 0; e < n; ++e) {
        const double ax = (double)__uint_as_float(w[e] & 0x7FFFFFFFu);
        if (ax != 0.0) dp += ax * exp2(L + b * log2(ax));
    }
    return dp;
}

// Adds the counted symbols to the current histogram and empties the table.
__device__ void flush_counts(Smem &sm, uint64_t *clamped, int hid)
{
    // (callers synchronise before: all counting under the old key is complete)
    const int qmin = sm.cold.qmin, qmax = sm.cold.qmax;
    unsigned long long *cl = reinterpret_cast<unsigned long long *>(clamped);
    auto add = [&](int q, uint32_t n) {
        if (q < qmin) { q = qmin; atomicAdd(&sm.clampc[0], n); }
        else if (q > qmax) { q = qmax; atomicAdd(&sm.clampc[1], n); }
        atomicAdd(&sm.cold.row[q - qmin], (unsigned long long)n);
    };
    if (sm.cold.rows_mode) {
        const int lane = threadIdx.x & 31;
        for (uint32_t r0 = threadIdx.x >> 5; r0 < kSymCells + 2; r0 += kWarps) {
            const uint32_t row = (r0 + blockIdx.x * 13u) % (kSymCells + 2);   // (CTAs start at different rows)
            const uint32_t v = sm.cnt[row * 32 + lane];
            const uint32_t n = __reduce_add_sync(0xFFFFFFFFu, v);
            if (n != 0u) {
                sm.cnt[row * 32 + lane] = 0u;
                if (lane == 0 && row >= 1 && row <= kSymCells) add((int)row - 1 - (int)(kSymCells / 2), n);
            }
        }
    } else {
        for (uint32_t i = threadIdx.x; i < kWinCells + 2; i += kThreads) {
            const uint32_t c = (i + blockIdx.x * 61u) % (kWinCells + 2);
            const uint32_t n = sm.cnt[c];
            if (n != 0u) {
                sm.cnt[c] = 0u;
                if (c >= 1 && c <= kWinCells) add((int)c - 1 - (int)(kWinCells / 2), n);
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < 2) {
        const uint32_t n = sm.clampc[threadIdx.x];
        if (n != 0u && cl != nullptr) atomicAdd(cl + 2 * hid + threadIdx.x, (unsigned long long)n);
        sm.clampc[threadIdx.x] = 0u;
    }
    __syncthreads();
}

// Eight gradient values to g (16-byte aligned; `wide`: 32-byte aligned, one 256-bit store per thread).
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

// n (<= 8) elements held in two vectors: the branch-free pass, the fix-up if one is needed, the
// penalty partial.  Returns through g.
template <int FLAGS, int MODE>
__device__ __forceinline__ void process8(const uint4 &lo, const uint4 &hi, int n, float (&g)[8], const Lane &ln, Smem &sm,
                                         Acc &acc, uint32_t (&clampc)[2])
{
    constexpr bool MOM = (FLAGS & kMoments) != 0, GRAD = (FLAGS & kGrad) != 0, HIST = (FLAGS & kHist) != 0;
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    float mp = 0.0f, anyt = 0.0f, m1 = 0.0f, m2 = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (i < n) g[i] = one_elem<FLAGS, MODE>(w[i], ln, mp, anyt, m1, m2, acc);
    }
    const bool grad_bad = GRAD && !(mp <= FLT_MAX);
    if (grad_bad || (HIST && count_miss<MODE>(anyt))) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (i < n) g[i] = fix_elem<FLAGS, MODE>(w[i], g[i], grad_bad, ln, sm, clampc);
        }
    }
    if constexpr (MOM) {
        if (run_sums_exact_enough(m1, m2)) {
            acc.s1 += (double)m1;
            acc.s2 += (double)m2;
        } else {     // a square or a sum outside the fp32 range, or an inf or nan entry: these elements again in fp64
            for (int e = 0; e < n; ++e) {
                const uint32_t ab = w[e] & 0x7FFFFFFFu;
                if (ab < 0x7F800000u) {
                    const double ax = (double)__uint_as_float(ab);
                    acc.s1 += ax;
                    acc.s2 += ax * ax;
                } else {
                    acc.bad += 1u;
                }
            }
        }
    }
    if constexpr (GRAD && (FLAGS & kEg) == 0) {
        // a product or a gradient that left the fp32 range, or a NaN marker, sends the vector to fp64
        if (mp <= FLT_MAX) acc.pen += (double)mp;
        else acc.pen += pen_exact(lo, hi, n, sm.cold.L, sm.cold.b, sm.cold.active);
    }
}

// One contiguous run of n elements: scalar head up to the first 16-byte boundary of x, pairs of
// 128-bit vectors through the asynchronous-copy ring, scalar tail.  If the gradient's address is not
// 16-byte aligned at the same element the whole run is scalar.
template <typename TG, int FLAGS, int MODE>
__device__ __forceinline__ void process_range(const float *x, TG *gout, int64_t n, bool accumulate, const Lane &ln,
                                              Smem &sm, Acc &acc, uint32_t (&clampc)[2])
{
    constexpr bool GRAD = (FLAGS & kGrad) != 0;
    const int tid = threadIdx.x;
    int64_t head = (int64_t)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / 4u);
    head = min(head, n);
    if (gout != nullptr && (reinterpret_cast<uintptr_t>(gout + head) & 15u) != 0) head = n;
    // (the body starts a block of the gradient, or of x when there is none: what a warp moves per step)
    else head = aligned_head(head, n, reinterpret_cast<uintptr_t>(x), reinterpret_cast<uintptr_t>(gout), 4u, (unsigned)sizeof(TG),
                             gout != nullptr ? 256u * (unsigned)sizeof(TG) : 1024u);
    const int64_t nvec = (n - head) / 8;          // units of eight elements
    const int64_t tail0 = head + nvec * 8;

    for (int64_t i = tid; i < head + (n - tail0); i += kThreads) {
        const int64_t idx = i < head ? i : tail0 + (i - head);
        if (!GG_IN_BOUNDS(idx, n)) continue;
        float g[8];
        process8<FLAGS, MODE>(make_uint4(__float_as_uint(__ldg(x + idx)), 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u), 1, g, ln,
                              sm, acc, clampc);
        if constexpr (GRAD) {
            if (gout != nullptr) {
                float v = g[0];
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

    // (a CTA's run never exceeds device memory / grid size elements: 32-bit unit indices suffice)
    // Each thread owns slot [d][.][tid] of every stage d: it fills it with two asynchronous 16-byte
    // copies (one commit group per iteration, empty past the end so that the group count stays in step)
    // and reads it back once the group that filled it has landed.
    const uint4 *xv = reinterpret_cast<const uint4 *>(x + head) + 2 * tid;
    TG *gv = gout != nullptr ? gout + head + (int64_t)tid * 8 : nullptr;
    const bool wide = (reinterpret_cast<uintptr_t>(gv) & 31u) == 0;
    const int nv = (int)nvec;
    const uint32_t slot0 = (uint32_t)__cvta_generic_to_shared(&sm.stage[0][0][tid]);
    constexpr uint32_t kHalfBytes = sizeof(uint4) * kThreads;        // from vector 0 to vector 1 of a slot
    constexpr uint32_t kStageBytes = 2 * kHalfBytes;
    auto fill = [&](uint32_t slot, const uint4 *src) {
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot), "l"(src) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot + kHalfBytes), "l"(src + 1) : "memory");
    };
#pragma unroll
    for (int d = 0; d < kDepth - 1; ++d) {
        if (tid + d * kThreads < nv && GG_IN_BOUNDS(head + (int64_t)(tid + d * kThreads) * 8 + 7, n)) fill(slot0 + d * kStageBytes, xv + 2 * d * kThreads);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    uint32_t rd = 0, wr = (kDepth - 1) * kStageBytes;      // byte offsets of the slot to read / to fill next
    for (int v = tid; v < nv; v += kThreads) {
        // fill the slot emptied by the previous iteration (its values are in registers since then)
        if (v + (kDepth - 1) * kThreads < nv && GG_IN_BOUNDS(head + (int64_t)(v + (kDepth - 1) * kThreads) * 8 + 7, n))
            fill(slot0 + wr, xv + 2 * (kDepth - 1) * kThreads);
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group %0;" ::"n"(kDepth - 1) : "memory");
        uint4 lo, hi;
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w) : "r"(slot0 + rd) : "memory");
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w) : "r"(slot0 + rd + kHalfBytes) : "memory");
        float g[8];
        process8<FLAGS, MODE>(lo, hi, 8, g, ln, sm, acc, clampc);
        if constexpr (GRAD) {
            if (gv != nullptr && GG_IN_BOUNDS(head + (int64_t)v * 8 + 7, n)) store8<TG>(gv, g, accumulate, wide);
        }
        rd = rd + kStageBytes == kDepth * kStageBytes ? 0u : rd + kStageBytes;
        wr = wr + kStageBytes == kDepth * kStageBytes ? 0u : wr + kStageBytes;
        xv += 2 * kThreads;
        if (gv != nullptr) gv += kThreads * 8;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

template <typename TG, int FLAGS>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) tail_f32_kernel(const StreamArgs a)
{
    constexpr bool MOM = (FLAGS & kMoments) != 0, GRAD = (FLAGS & kGrad) != 0, HIST = (FLAGS & kHist) != 0;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // contiguous range of tiles for this CTA
    const int64_t nt = a.map.n_tiles;
    const int t_begin = (int)(nt * blockIdx.x / gridDim.x);
    const int t_end = (int)(nt * (blockIdx.x + 1) / gridDim.x);

    if constexpr (HIST) {
        for (int i = tid; i < (int)kCntWords; i += kThreads) sm.cnt[i] = 0u;
        if (tid < 2) sm.clampc[tid] = 0u;
    }
    if (tid == 0) { sm.cold.active = 0; sm.cold.sign_flip = 0u; sm.cold.rows_mode = 0; sm.cold.L = 0.0; sm.cold.b = 0.0; }
    if (tid < 128) sm.lg[tid] = log2(1.0 + (double)tid * (1.0 / 128.0));
    int cur_hid = -1, cur_mode = kModeWords;
    uint32_t cur_inv_bits = 0;
    bool have_key = false;
    const bool accumulate = GRAD && a.accumulate != 0;
    const uint32_t cnt_addr = (uint32_t)__cvta_generic_to_shared(sm.cnt);
    Lane ln{};
    ln.b_addr = (uint32_t)__cvta_generic_to_shared(sm.brep) + (uint32_t)lane * 4u;
    __syncthreads();

    for (int t = t_begin; t < t_end;) {
        // ---- one run: the tiles of this CTA's range that lie in segment s
        const int s = a.map.tile_seg[t];
        const int64_t len = a.map.seg_len[s];
        const int t_first = a.map.tile_prefix[s];
        const int t_stop = min(t_end, a.map.tile_prefix[s + 1]);
        const int64_t off = (int64_t)(t - t_first) * kTile;
        const int64_t n = min(len, (int64_t)(t_stop - t_first) * kTile) - off;
        const float *x = reinterpret_cast<const float *>(a.map.seg_ptr[s]) + off;
        int mode = kModeWords;

        if constexpr (GRAD && (FLAGS & kEg) != 0) {
            // code-length gradient: one factor per segment (Eq. 7 relaxed), no tables
            const float inv_s = (float)(1.0 / (double)a.step[s]);
            ln.eg_c = (float)(a.lambda * 4.0 * (double)inv_s / ((double)len * 0.6931471805599453094));
            ln.eg_two_k = 1u << a.eg_k;
            ln.qmin = a.qmin;
            ln.qmax = a.qmax;
        } else if constexpr (GRAD) {
            const double beta = a.beta[s], alpha = a.alpha[s];
            const double lam = a.mean_reduction ? a.lambda / (double)len : a.lambda;
            const bool active = (beta > 0.0) && (alpha > 0.0) && (lam != 0.0) && (lam == lam);
            const double b = beta - 1.0;
            const double L = active ? log2(fabs(lam) * beta) - beta * log2(alpha) : 0.0;
            if (tid == 0) {
                sm.cold.b = b;
                sm.cold.L = L;
                sm.cold.sign_flip = lam < 0.0 ? 0x80000000u : 0u;
                sm.cold.active = active;
            }
            if (tid < 256) {
                // One factor serves exponent k if |L + b (k-127)| <= 100 (its product with B, at most 2^2
                // either way, and with the series stays normal) and the series applies (|b| <= 2).
                // Zero/subnormal (k = 0) and inf/nan (k = 255) get the marker.  Without a gradient all is zero.
                float one = 0.0f;
                if (active) {
                    const double e0 = L + b * (double)(tid - 127);
                    const bool ok = tid >= 1 && tid <= 254 && fabs(e0) <= 100.0 && fabs(b) <= 2.0;
                    one = ok ? (float)(lam < 0.0 ? -exp2_short(e0) : exp2_short(e0)) : __int_as_float(0x7FC00000);
                }
                s_a1[tid] = one;
            } else if (tid < 384) {
                const int j = tid - 256;
                sm.B[j] = active ? (float)exp2_short(b * sm.lg[j]) : 1.0f;
            }
            __syncthreads();
            for (int i = tid; i < 128 * 32; i += kThreads) sm.brep[i] = sm.B[i >> 5];      // B[j] into every bank of row j
            const float bf = (float)b;
            ln.c1 = bf;
            ln.c2 = ln.c1 * (bf - 1.0f) * 0.5f;
            ln.c3 = ln.c2 * (bf - 2.0f) * (1.0f / 3.0f);
            ln.c4 = ln.c3 * (bf - 3.0f) * 0.25f;
        }
        if constexpr (HIST) {
            const int hid = a.map.hist_id ? a.map.hist_id[s] : s;
            const float step = a.step[s];
            const float inv = (float)(1.0 / (double)step);
            __syncthreads();
            double sd = 0.0;
            if (a.seg_sd != nullptr) {
                sd = a.seg_sd[s];
            } else {
                // The scale of the data is taken from the first elements of the run (one per thread):
                // it only decides how the counts are laid out, never what is counted.
                const int m = (int)min(n, (int64_t)kThreads);
                float ss = 0.0f;
                for (int i = tid; i < m; i += kThreads) {
                    const float v = __ldg(x + i);
                    if (fabsf(v) <= 1e18f) ss = fmaf(v, v, ss);        // (inf, nan and values whose squares overflow are left out)
                }
                const double ws = warp_sum((double)ss);
                if ((tid & 31) == 0) sm.red[2][tid >> 5] = ws;          // (free here: the barrier above follows the run before)
                __syncthreads();
                double tot = 0.0;
                for (int w = 0; w < kWarps; ++w) tot += sm.red[2][w];
                sd = m > 0 ? sqrt(tot / (double)m) : 0.0;
                __syncthreads();
            }
            // rows when the scale of the data is known and the row window reaches 6.5 standard deviations
            if (sd > 0.0 && step > 0.0f && (double)(kSymCells / 2) * (double)step >= 6.5 * sd && inv < 3.0e38f) mode = kModeRows;
            const bool same_key = have_key && hid == cur_hid && __float_as_uint(inv) == cur_inv_bits && mode == cur_mode;
            if (!same_key) {
                if (have_key) flush_counts(sm, a.clamped, cur_hid);
                have_key = true;
                cur_hid = hid;
                cur_inv_bits = __float_as_uint(inv);
                cur_mode = mode;
                if (tid == 0) {
                    sm.cold.inv = inv;
                    sm.cold.qmin = a.qmin;
                    sm.cold.qmax = a.qmax;
                    sm.cold.row = reinterpret_cast<unsigned long long *>(a.hist) +
                                  (int64_t)hid * ((int64_t)a.qmax - (int64_t)a.qmin + 1);
                    sm.cold.rows_mode = mode == kModeRows;
                }
            }
            ln.inv = inv;
            // symbol floor(t) counts at cnt + (floor(t) + half + 1) * bytes-per-symbol (+ the lane's word in a
            // row); one_elem adds the bits of floor(t) + magic shifted by the same amount (mod 2^32)
            if (mode == kModeRows) ln.c_addr = cnt_addr + (uint32_t)lane * 4u + ((kSymCells / 2 + 1 - kMagicBits) << 7);
            else ln.c_addr = cnt_addr + ((kWinCells / 2 + 1 - kMagicBits) << 2);
        }
        __syncthreads();

        // ---- stream the run
        TG *gout = nullptr;
        if constexpr (GRAD) {
            if (a.map.grad_ptr != nullptr) gout = reinterpret_cast<TG *>(a.map.grad_ptr[s]) + off;
        }
        Acc acc;
        uint32_t clampc[2] = {0u, 0u};
        if (HIST && mode == kModeRows) process_range<TG, FLAGS, kModeRows>(x, gout, n, accumulate, ln, sm, acc, clampc);
        else process_range<TG, FLAGS, kModeWords>(x, gout, n, accumulate, ln, sm, acc, clampc);

        // ---- per-run results: the partial sums in a fixed order (butterfly, then the warps in sequence) to the
        // slot of the run's first tile, zeros to its other tiles; clamp counts
        if constexpr (MOM) {
            const double w1 = warp_sum(acc.s1), w2 = warp_sum(acc.s2);
            const uint32_t wb = __reduce_add_sync(0xFFFFFFFFu, acc.bad);
            float wmin = acc.xmin, wmax = acc.xmax;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                wmin = fminf(wmin, __shfl_xor_sync(0xFFFFFFFFu, wmin, o));
                wmax = fmaxf(wmax, __shfl_xor_sync(0xFFFFFFFFu, wmax, o));
            }
            if (lane == 0) { sm.red[0][warp] = w1; sm.red[1][warp] = w2; sm.bad[warp] = wb; sm.mn[warp] = wmin; sm.mx[warp] = wmax; }
        }
        if constexpr (GRAD) {
            const double wp = warp_sum(acc.pen);
            if (lane == 0) sm.red[2][warp] = wp;
        }
        if constexpr (HIST) {
            if (clampc[0]) atomicAdd(&sm.clampc[0], clampc[0]);
            if (clampc[1]) atomicAdd(&sm.clampc[1], clampc[1]);
        }
        __syncthreads();
        if constexpr (MOM || GRAD) {
            for (int tt = t + 1 + tid; tt < t_stop; tt += kThreads) {
                if constexpr (MOM) {
                    a.part.s1[tt] = 0.0; a.part.s2[tt] = 0.0; a.part.bad[tt] = 0u;
                    a.part.xmin[tt] = INFINITY; a.part.xmax[tt] = -INFINITY;
                }
                if constexpr (GRAD) a.part.pen[tt] = 0.0;
            }
            if (tid == 0) {
                if constexpr (MOM) {
                    double r1 = 0.0, r2 = 0.0;
                    uint32_t rb = 0;
                    float rmin = INFINITY, rmax = -INFINITY;
                    for (int w = 0; w < kWarps; ++w) {
                        r1 += sm.red[0][w]; r2 += sm.red[1][w]; rb += sm.bad[w];
                        rmin = fminf(rmin, sm.mn[w]); rmax = fmaxf(rmax, sm.mx[w]);
                    }
                    a.part.s1[t] = r1; a.part.s2[t] = r2; a.part.bad[t] = rb;
                    a.part.xmin[t] = rmin; a.part.xmax[t] = rmax;
                }
                if constexpr (GRAD) {
                    double rp = 0.0;
                    for (int w = 0; w < kWarps; ++w) rp += sm.red[2][w];
                    a.part.pen[t] = sm.cold.sign_flip ? -rp : rp;     // the penalty carries lambda's sign
                }
            }
            __syncthreads();
        }
        t = t_stop;
    }
    if constexpr (HIST) {
        if (have_key) flush_counts(sm, a.clamped, cur_hid);
    }
}

template <typename TG, int FLAGS>
cudaError_t launch_one(const StreamArgs &a, int sm_count, cudaStream_t st)
{
    auto kern = tail_f32_kernel<TG, FLAGS>;
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

}  // namespace

cudaError_t launch_tail_f32(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a, int sm_count,
                            cudaStream_t st)
{
    if (a.map.n_tiles <= 0) return cudaSuccess;
    if (has_grad_out && grad_dtype == GG_BF16) return launch_typed<uint16_t>(flags, a, sm_count, st);
    return launch_typed<float>(flags, a, sm_count, st);
}

}  // namespace gg
