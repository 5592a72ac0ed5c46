// The whole pass for short bf16 segments (per-token activation rows and the like): one warp per
// segment.  The warp reads its segment once for the moments, inverts the moment ratio itself,
// builds the segment's two gradient tables, and reads the segment a second time, while it is
// still in L1/L2, for the gradient and the histogram.  DRAM sees the input once and the gradient
// once; nothing is staged between kernels and no per-tile scratch is used.
//
//   * fit: beta and alpha come from a table of ln rho and ln(alpha/sigma) over a grid of ln beta
//     (built once per context) by cubic interpolation: no lgamma at fit time.
//   * gradient: |g| = A[e] * B[j] as in the long-segment kernel, with per-warp tables: A for the 64
//     exponents around the segment's scale as one fp32 factor, NaN elsewhere; a NaN sends the
//     element to the fp64 evaluation, which also adds its penalty term in fp64.
//   * histogram: a CTA-wide pattern-count table serves the segments whose histogram and step equal
//     those of the CTA's first segment (the common case: many rows, one histogram); other segments
//     add to global memory element by element.
#include <cuda_bf16.h>
#include <float.h>

#include "gg_fit_table.cuh"
#include "gg_device.cuh"
#include "gg_internal.h"
#include "gg_small_common.cuh"

namespace gg {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kCtasPerSm = 2;
constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kTabExp = 64;          // exponents around the segment's scale whose A is evaluated
struct WarpTab {
    float a1[256];       // A[e] as one factor (with lambda's sign); NaN where that is not possible or not evaluated
    float B[128];
};

struct Smem {
    // cell p * 2 + sign: magnitude pattern c_base + p; then the sentinel pair; then the values below the
    // window (all of symbol 0, or -1 if negative) when the window starts at or below one step
    uint32_t cnt[kCells];
    WarpTab tab[kWarps];
    double log2m[128];                 // log2(1 + j/128): the same for every segment
    // the CTA's histogram key
    int key_hid;
    uint32_t key_inv_bits;
    uint32_t c_base;
    int key_on;
    int below_ok;                      // values below the window quantise to 0 / -1
};

__device__ __forceinline__ double log_rho(double beta)
{
    return 2.0 * lgamma(2.0 / beta) - lgamma(1.0 / beta) - lgamma(3.0 / beta);
}

__global__ void seed_table_kernel(double *table)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i > kSeedCells) return;
    const double lo = log(GG_BETA_LO), hi = log(GG_BETA_HI);
    const double beta = exp(lo + (hi - lo) * ((double)i / (double)kSeedCells));
    table[i] = log_rho(beta);
    table[kSeedCells + 1 + i] = 0.5 * (lgamma(1.0 / beta) - lgamma(3.0 / beta));
}

template <typename TG>
__device__ __forceinline__ float load_grad(const TG *g)
{
    if constexpr (sizeof(TG) == 4) return *g;
    else return __uint_as_float((uint32_t)*g << 16);
}

template <typename TG>
__device__ __forceinline__ void store_grad(TG *g, float v)
{
    if constexpr (sizeof(TG) == 4) *g = v;
    else *g = __bfloat16_as_ushort(__float2bfloat16_rn(v));
}

// Per-segment constants of the second pass.
struct SegConst {
    double L, b;
    bool active;
    uint32_t sign_flip;
    int e_lo;             // first exponent of the warp's A table
    // histogram
    bool hist, fast;      // fast: the CTA table serves this segment
    float inv;
    int32_t qmin, qmax;
    unsigned long long *row;
    uint32_t c_base;
    bool below_ok;
};

// One element of a 32-bit word w holding two bf16 values (HALF 0: low half, 1: high half).  Branch
// free.  Gradient: a NaN entry of the warp's A table makes the vector's penalty partial NaN, which
// the caller checks once per vector.  Count (HIST 1: the CTA table serves the segment): `anyc` keeps
// the largest window index so that one compare per vector finds values outside the window; those
// count in the sentinel cells.  HIST 2 (the table does not serve the segment) counts in global memory.
template <bool GRAD, int HIST, int HALF>
__device__ __forceinline__ float small_elem(uint32_t w, const SegConst &k, uint32_t a_addr, uint32_t b_addr, uint32_t cnt_addr,
                                            float &mp, uint32_t &anyc, uint32_t (&clampc)[2])
{
    const uint32_t xb = HALF ? (w & 0xFFFF0000u) : (w << 16);
    float g = 0.0f;
    if constexpr (GRAD) {
        const uint32_t e4 = HALF ? ((w >> 21) & 0x3FCu) : ((w >> 5) & 0x3FCu);     // exponent field * 4
        const uint32_t j4 = HALF ? ((w >> 14) & 0x1FCu) : ((w << 2) & 0x1FCu);     // mantissa bits * 4
        const float ga = lds_f32(a_addr + e4) * lds_f32(b_addr + j4);
        mp = fmaf(fabsf(__uint_as_float(xb)), fabsf(ga), mp);
        g = __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));
    }
    if constexpr (HIST == 1) {
        const uint32_t mag = HALF ? ((w >> 16) & 0x7FFFu) : (w & 0x7FFFu);
        uint32_t p = mag - k.c_base;
        anyc = max(anyc, p);
        p = min(p, kCntPat);
        const uint32_t sign4 = HALF ? ((w >> 29) & 4u) : ((w >> 13) & 4u);
        red_inc(cnt_addr + p * 8u + sign4);
    } else if constexpr (HIST == 2) {
        const int c = count_global(xb, k.inv, k.qmin, k.qmax, k.row);
        if (c) clampc[c - 1] += 1u;
    }
    return g;
}

// Redo of whatever part of an element (fp32 bits) the branch-free path could not do; g is its
// gradient from the first pass.  grad_bad: the vector's penalty partial is not a finite number, so
// the whole vector's penalty terms are added here instead, in fp64.
template <bool GRAD, int HIST>
__device__ __forceinline__ float small_fix(uint32_t xb, float g, bool grad_bad, const SegConst &k, const WarpTab &tab, Smem &sm,
                                           double &pen, uint32_t (&clampc)[2])
{
    const uint32_t mag = (xb & 0x7FFFFFFFu) >> 16;
    if constexpr (GRAD) {
        if (grad_bad) {
            const float a = tab.a1[mag >> 7];
            const double ax = (double)__uint_as_float(mag << 16);
            if (a != a) {     // this element read a NaN marker: the fp64 evaluation
                const double gd = grad_fp64(mag, k.L, k.b, k.active);
                pen += ax * gd;
                g = __uint_as_float(__float_as_uint((float)gd) ^ k.sign_flip ^ (xb & 0x80000000u));
            } else {
                pen += ax * (double)fabsf(g);
            }
        }
    }
    if constexpr (HIST == 1) {
        if (mag - k.c_base >= kCntPat) {
            if (k.below_ok && mag < k.c_base) {
                atomicAdd(&sm.cnt[kBelow + (mag != 0u ? (xb >> 31) : 0u)], 1u);
            } else {
                const int c = count_global(xb, k.inv, k.qmin, k.qmax, k.row);
                if (c) clampc[c - 1] += 1u;
            }
        }
    }
    return g;
}

// Second pass over one segment by one warp.
template <typename TG, bool GRAD, int HIST>
__device__ __forceinline__ void second_pass(const SmallArgs &a, int s, const uint16_t *x, TG *gout, int head, int nvec,
                                            int tail0, int n_scalar, double beta, const SegConst &k, const WarpTab &tab,
                                            Smem &sm)
{
    if constexpr (!GRAD && HIST == 0) return;     // a fit-only call has no second pass
    const int lane = threadIdx.x & 31;
    const uint4 *xv = reinterpret_cast<const uint4 *>(x + head);
    double pen = 0.0;
    uint32_t clampc[2] = {0u, 0u};
    const bool accumulate = GRAD && a.accumulate != 0;
    // 32-bit shared addresses of the warp's tables and of the CTA's count cells
    const uint32_t a_addr = (uint32_t)__cvta_generic_to_shared(tab.a1), b_addr = (uint32_t)__cvta_generic_to_shared(tab.B);
    const uint32_t cnt_addr = (uint32_t)__cvta_generic_to_shared(sm.cnt);
    for (int i = lane; i < n_scalar; i += 32) {
        const int idx = i < head ? i : tail0 + (i - head);
        const uint32_t h = (uint32_t)__ldg(x + idx);
        float mp = 0.0f;
        uint32_t anyc = 0;
        float g = small_elem<GRAD, HIST, 0>(h, k, a_addr, b_addr, cnt_addr, mp, anyc, clampc);
        const bool grad_bad = GRAD && !(mp <= FLT_MAX);
        if (grad_bad || (HIST == 1 && anyc >= kCntPat)) g = small_fix<GRAD, HIST>(h << 16, g, grad_bad, k, tab, sm, pen, clampc);
        if constexpr (GRAD) {
            if (!grad_bad) pen += (double)mp;
            if (gout != nullptr) {
                if (accumulate) g += load_grad<TG>(gout + idx);
                store_grad<TG>(gout + idx, g);
            }
        }
    }
    // (loads run three vectors ahead of their use: the pass is bound by cache latency otherwise)
    uint4 q0 = make_uint4(0u, 0u, 0u, 0u), q1 = q0, q2 = q0;
    if (lane < nvec) q0 = __ldg(xv + lane);
    if (lane + 32 < nvec) q1 = __ldg(xv + lane + 32);
    if (lane + 64 < nvec) q2 = __ldg(xv + lane + 64);
    for (int v = lane; v < nvec; v += 32) {
        const uint4 raw = q0;
        q0 = q1;
        q1 = q2;
        if (v + 96 < nvec) q2 = __ldg(xv + v + 96);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
        float g[8];
        float mp = 0.0f;
        uint32_t anyc = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            g[2 * i] = small_elem<GRAD, HIST, 0>(w[i], k, a_addr, b_addr, cnt_addr, mp, anyc, clampc);
            g[2 * i + 1] = small_elem<GRAD, HIST, 1>(w[i], k, a_addr, b_addr, cnt_addr, mp, anyc, clampc);
        }
        // (table products are normal numbers whose terms |x| |g| stay far inside the fp32 range, so a
        // partial that is not finite means a NaN marker was read)
        const bool grad_bad = GRAD && !(mp <= FLT_MAX);
        if (grad_bad || (HIST == 1 && anyc >= kCntPat)) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t xb = (i & 1) ? (w[i >> 1] & 0xFFFF0000u) : (w[i >> 1] << 16);
                g[i] = small_fix<GRAD, HIST>(xb, g[i], grad_bad, k, tab, sm, pen, clampc);
            }
        }
        if constexpr (GRAD) {
            if (!grad_bad) pen += (double)mp;
            if (gout != nullptr) {
                TG *gp = gout + head + v * 8;
                if constexpr (sizeof(TG) == 4) {
                    float4 *p4 = reinterpret_cast<float4 *>(gp);
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        float4 o = make_float4(g[4 * q], g[4 * q + 1], g[4 * q + 2], g[4 * q + 3]);
                        if (accumulate) {
                            const float4 old = p4[q];
                            o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                        }
                        __stcs(p4 + q, o);
                    }
                } else {
                    uint32_t o[4];
                    const uint32_t *p1 = reinterpret_cast<const uint32_t *>(gp);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float lo = g[2 * q], hi = g[2 * q + 1];
                        if (accumulate) {
                            const uint32_t old = p1[q];
                            lo += __uint_as_float(old << 16);
                            hi += __uint_as_float(old & 0xFFFF0000u);
                        }
                        o[q] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) |
                               ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
                    }
                    __stcs(reinterpret_cast<uint4 *>(gp), make_uint4(o[0], o[1], o[2], o[3]));
                }
            }
        }
    }
    if constexpr (GRAD) {
        pen = warp_sum(pen);
        if (lane == 0 && a.penalty) {
            // sum |x| |g| = |lambda| beta sum (|x|/alpha)^beta; the penalty carries lambda's sign
            a.penalty[s] = beta > 0.0 ? (k.sign_flip ? -pen : pen) / beta : 0.0;
        }
    }
    if constexpr (HIST != 0) {
        if (a.clamped != nullptr) {
            const uint32_t c0 = __reduce_add_sync(kFull, clampc[0]), c1 = __reduce_add_sync(kFull, clampc[1]);
            const int hid = a.map.hist_id ? a.map.hist_id[s] : s;
            if (lane == 0 && c0) atomicAdd(reinterpret_cast<unsigned long long *>(a.clamped) + 2 * hid, (unsigned long long)c0);
            if (lane == 0 && c1) atomicAdd(reinterpret_cast<unsigned long long *>(a.clamped) + 2 * hid + 1, (unsigned long long)c1);
        }
    }
}

template <typename TG, bool GRAD, bool HIST>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) small_bf16_kernel(const SmallArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_seg = a.map.n_seg;
    const int64_t n_bins = (int64_t)a.qmax - (int64_t)a.qmin + 1;

    if constexpr (HIST) {
        for (int i = tid; i < (int)kCells; i += kThreads) sm.cnt[i] = 0u;
    }
    if (tid < 128) sm.log2m[tid] = log2(1.0 + (double)tid * (1.0 / 128.0));
    if (tid == 0) {
        // the CTA's histogram key: that of the first segment it handles, when steps are given
        sm.key_on = 0;
        const int s0 = blockIdx.x * kWarps;
        if (HIST && a.do_hist && !a.step_from_alpha && s0 < n_seg) {
            const float step = a.step[s0];
            sm.key_hid = a.map.hist_id ? a.map.hist_id[s0] : s0;
            sm.key_inv_bits = __float_as_uint((float)(1.0 / (double)step));
            const int e_top = window_top_exponent((double)step);
            sm.c_base = (uint32_t)(e_top - (kCntBinades - 1)) << 7;
            // the window starts 2^-4 steps up unless its position had to be clamped
            sm.below_ok = step > 0.0f && e_top == ilogb((double)step) + 127 + 11;
            sm.key_on = 1;
        }
    }
    __syncthreads();
    WarpTab &tab = sm.tab[warp];

    for (int s = blockIdx.x * kWarps + warp; s < n_seg; s += gridDim.x * kWarps) {
        const uint16_t *x = reinterpret_cast<const uint16_t *>(a.map.seg_ptr[s]);
        const int len = (int)a.map.seg_len[s];
        TG *gout = nullptr;
        if constexpr (GRAD) {
            if (a.map.grad_ptr != nullptr) gout = reinterpret_cast<TG *>(a.map.grad_ptr[s]);
        }
        // scalar head up to the first 16-byte boundary of x, 128-bit vector body, scalar tail; if the
        // gradient is not 16-byte aligned at the same element the whole segment is scalar
        int head = (int)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / 2u);
        head = min(head, len);
        if (gout != nullptr && (reinterpret_cast<uintptr_t>(gout + head) & 15u) != 0) head = len;
        const int nvec = (len - head) / 8;
        const int tail0 = head + nvec * 8;
        const int n_scalar = head + (len - tail0);
        const uint4 *xv = reinterpret_cast<const uint4 *>(x + head);

        // ---- first pass: moments (fp32 runs of 8, then fp64), extremes, non-finite count
        double s1 = 0.0, s2 = 0.0;
        uint32_t bad = 0;
        float xmin = INFINITY, xmax = -INFINITY;
        for (int i = lane; i < n_scalar; i += 32) {
            const int idx = i < head ? i : tail0 + (i - head);
            const uint32_t xb = (uint32_t)__ldg(x + idx) << 16;
            const uint32_t am = xb & 0x7FFFFFFFu;
            if (am < 0x7F800000u) { s1 += (double)__uint_as_float(am); s2 += (double)__uint_as_float(am) * (double)__uint_as_float(am); }
            else bad += 1u;
            xmin = fminf(xmin, __uint_as_float(xb));
            xmax = fmaxf(xmax, __uint_as_float(xb));
        }
        // extremes of the vector body as packed bf16 (even and odd elements); the padding of a ragged trip is
        // guarded below, so no zero enters them
        __nv_bfloat162 mn2 = __floats2bfloat162_rn(INFINITY, INFINITY), mx2 = __floats2bfloat162_rn(-INFINITY, -INFINITY);
        for (int v0 = lane; v0 < nvec; v0 += 128) {
            // four independent loads per trip
            uint4 r4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                r4[u] = make_uint4(0u, 0u, 0u, 0u);      // (zeros add nothing to the sums or the extremes' validity)
                if (v0 + 32 * u < nvec) r4[u] = __ldg(xv + v0 + 32 * u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
            if (v0 + 32 * u >= nvec) break;
            const uint4 raw = r4[u];
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
            float m1 = 0.0f, m2 = 0.0f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                // both elements of a word at once; an inf or nan makes the sums inf or nan, and the vector is then
                // summed again element by element below, where it is counted and left out
                const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
                m1 += fabsf(lo);
                m1 += fabsf(hi);
                m2 = fmaf(lo, lo, m2);
                m2 = fmaf(hi, hi, m2);
                const __nv_bfloat162 pr = *reinterpret_cast<const __nv_bfloat162 *>(&w[i]);
                mn2 = __hmin2(mn2, pr);      // return the non-NaN operand, like fminf
                mx2 = __hmax2(mx2, pr);
            }
            if (run_sums_exact_enough(m1, m2)) {
                s1 += (double)m1;
                s2 += (double)m2;
            } else {     // a square or a sum left the fp32 range: this vector again in fp64
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint32_t am = ((i & 1) ? (w[i >> 1] & 0xFFFF0000u) : (w[i >> 1] << 16)) & 0x7FFFFFFFu;
                    if (am < 0x7F800000u) {
                        const double ax = (double)__uint_as_float(am);
                        s1 += ax;
                        s2 += ax * ax;
                    } else {
                        bad += 1u;
                    }
                }
            }
            }
        }
        xmin = fminf(xmin, fminf(__low2float(mn2), __high2float(mn2)));
        xmax = fmaxf(xmax, fmaxf(__low2float(mx2), __high2float(mx2)));
        s1 = warp_sum(s1);
        s2 = warp_sum(s2);
        bad = __reduce_add_sync(kFull, bad);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            xmin = fminf(xmin, __shfl_xor_sync(kFull, xmin, o));
            xmax = fmaxf(xmax, __shfl_xor_sync(kFull, xmax, o));
        }

        // ---- fit (every lane holds the same values)
        uint32_t flags = bad ? GG_FLAG_NONFINITE : 0u;
        double beta = 0.0, alpha = 0.0;
        if (len <= 0 || !(s2 > 0.0)) {
            flags |= GG_FLAG_DEGENERATE;
        } else {
            double m1 = s1 / (double)len, m2 = s2 / (double)len;
            double log_r = log(m1 * m1 / m2);
            if (log_r > kCarefulLogRatio && len <= kCarefulLen) {      // (an ill-conditioned fit: the sums again in fp64)
                careful_sums(a.map.seg_ptr[s], (int)GG_BF16, len, lane, s1, s2);
                m1 = s1 / (double)len;
                m2 = s2 / (double)len;
                log_r = log(m1 * m1 / m2);
            }
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
            alpha = sqrt(m2) * exp(lnz);       // Eq. 2 with sigma^2 = sum_sq / count
        }
        float step = 0.0f;
        if (HIST && a.do_hist) {
            step = a.step_from_alpha ? (float)(alpha * a.step_scale) : a.step[s];
            if (xmin <= xmax) {
                // the quantiser is monotone in x, so a symbol clamps iff one of the extremes does
                const float inv = (float)(1.0 / (double)step);
                const float tlo = __fmul_rn(xmin, inv), thi = __fmul_rn(xmax, inv);
                if ((double)floorf(tlo) < (double)a.qmin || (double)floorf(thi) > (double)a.qmax)
                    flags |= GG_FLAG_CLAMPED_SYMBOLS;
            }
        }
        if (lane == 0) {
            a.beta[s] = beta;
            a.alpha[s] = alpha;
            if (a.sum_abs) a.sum_abs[s] = s1;
            if (a.sum_sq) a.sum_sq[s] = s2;
            if (a.count) a.count[s] = len;
            if (a.flags) a.flags[s] = flags;
            if (HIST && a.do_hist && a.step_from_alpha && a.step_out) a.step_out[s] = step;
        }

        // ---- constants and tables of the second pass
        SegConst k{};
        if constexpr (GRAD) {
            const double lam = a.mean_reduction ? a.lambda / (double)max(len, 1) : a.lambda;
            k.active = (beta > 0.0) && (alpha > 0.0) && (lam != 0.0) && (lam == lam);
            k.sign_flip = lam < 0.0 ? 0x80000000u : 0u;
            k.b = beta - 1.0;
            k.L = k.active ? log2(fabs(lam) * beta) - beta * log2(alpha) : 0.0;
            // the table's 64 exponents: 40 binades below the standard deviation's to 23 above
            int e_c = 127;
            if (k.active) e_c = ilogb(sqrt(s2 / (double)len)) + 127;
            k.e_lo = max(1, min(254 - (kTabExp - 1), e_c - 40));
            __syncwarp();       // the previous segment's second pass is done with the tables
            // A for the kTabExp exponents from 40 binades below the standard deviation's upwards, NaN for
            // the rest (zero/subnormal, inf/nan and far binades go to the fp64 evaluation)
            for (int e = lane; e < 256; e += 32) {
                float v = k.active ? __int_as_float(0x7FC00000) : 0.0f;
                if (k.active && (uint32_t)(e - k.e_lo) < (uint32_t)kTabExp) {
                    // one fp32 factor serves if |L + b (e-127)| <= 100: its product with B stays a normal
                    // number; the same bound on L + beta (e-127) keeps the penalty terms |x| |g| normal too
                    const double de = (double)(e - 127);
                    const double e0 = k.L + k.b * de;
                    if (fabs(e0) <= 100.0 && fabs(e0 + de) <= 100.0) v = (float)(lam < 0.0 ? -exp2_short(e0) : exp2_short(e0));
                }
                tab.a1[e] = v;
            }
#pragma unroll
            for (int j = lane; j < 128; j += 32) tab.B[j] = k.active ? (float)exp2_short(k.b * sm.log2m[j]) : 1.0f;
            __syncwarp();
        }
        if constexpr (HIST) {
            k.hist = a.do_hist != 0;
            if (k.hist) {
                const int hid = a.map.hist_id ? a.map.hist_id[s] : s;
                k.inv = (float)(1.0 / (double)step);
                k.qmin = a.qmin;
                k.qmax = a.qmax;
                k.row = reinterpret_cast<unsigned long long *>(a.hist) + (int64_t)hid * n_bins;
                k.fast = sm.key_on && hid == sm.key_hid && __float_as_uint(k.inv) == sm.key_inv_bits;
                k.c_base = sm.c_base;
                k.below_ok = sm.below_ok != 0;
            }
        }

        // ---- second pass: gradient, penalty partial, counts (the segment is in L1/L2 now)
        if constexpr (HIST) {
            if (!k.hist) second_pass<TG, GRAD, 0>(a, s, x, gout, head, nvec, tail0, n_scalar, beta, k, tab, sm);
            else if (k.fast) second_pass<TG, GRAD, 1>(a, s, x, gout, head, nvec, tail0, n_scalar, beta, k, tab, sm);
            else second_pass<TG, GRAD, 2>(a, s, x, gout, head, nvec, tail0, n_scalar, beta, k, tab, sm);
        } else {
            second_pass<TG, GRAD, 0>(a, s, x, gout, head, nvec, tail0, n_scalar, beta, k, tab, sm);
        }
    }

    // ---- the CTA's pattern counts go to its slot of the scratch; small_flush_kernel turns them into
    // symbols.  (Adding them to the histogram from here would make every CTA hit the same few
    // thousand addresses with 64-bit atomics at the same time, which serialises.)
    if constexpr (HIST) {
        __syncthreads();
        uint32_t *slot = a.cta_counts + (size_t)blockIdx.x * kSmallSlotWords;
        for (uint32_t c = tid; c < kCells; c += kThreads) slot[c] = sm.key_on ? sm.cnt[c] : 0u;
        if (tid == 0) {
            slot[kCells + 0] = (uint32_t)sm.key_on;
            slot[kCells + 1] = (uint32_t)sm.key_hid;
            slot[kCells + 2] = sm.key_inv_bits;
            slot[kCells + 3] = sm.c_base;
        }
    }
}

template <typename TG>
cudaError_t launch_typed(const SmallArgs &a, int sm_count, cudaStream_t st)
{
    const int grid = small_grid(a.map.n_seg, sm_count);
    auto go = [&](auto kern) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem));
        if (e != cudaSuccess) return e;
        kern<<<grid, kThreads, sizeof(Smem), st>>>(a);
        return cudaGetLastError();
    };
    if (!a.do_hist) return a.do_grad ? go(small_bf16_kernel<TG, true, false>) : go(small_bf16_kernel<TG, false, false>);
    cudaError_t e = a.do_grad ? go(small_bf16_kernel<TG, true, true>) : go(small_bf16_kernel<TG, false, true>);
    if (e != cudaSuccess) return e;
    flush_slots_kernel<false><<<(kCells + 31) / 32, dim3(32, 8), 0, st>>>(a.cta_counts, grid, a.qmin, a.qmax, a.hist, a.clamped);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_small_bf16(gg_dtype grad_dtype, const SmallArgs &a, int sm_count, cudaStream_t st)
{
    if (a.map.n_seg <= 0) return cudaSuccess;
    if (a.do_grad && a.map.grad_ptr != nullptr && grad_dtype == GG_BF16) return launch_typed<uint16_t>(a, sm_count, st);
    return launch_typed<float>(a, sm_count, st);
}

cudaError_t launch_small_flush(const uint32_t *cta_counts, int n_slots, int32_t qmin, int32_t qmax, uint64_t *hist, uint64_t *clamped,
                               cudaStream_t st)
{
    if (n_slots <= 0) return cudaSuccess;
    if (n_slots > kMaxSlots) return cudaErrorInvalidValue;
    flush_slots_kernel<false><<<(kCells + 31) / 32, dim3(32, 8), 0, st>>>(cta_counts, n_slots, qmin, qmax, hist, clamped);
    return cudaGetLastError();
}

int small_grid(int32_t n_seg, int sm_count)
{
    return (int)min(min((int64_t)(n_seg + kWarps - 1) / kWarps, (int64_t)sm_count * kCtasPerSm), (int64_t)kMaxSlots);
}

cudaError_t launch_fit_seed_table(double *seed, cudaStream_t st)
{
    seed_table_kernel<<<(kSeedCells + 1 + 255) / 256, 256, 0, st>>>(seed);
    return cudaGetLastError();
}

}  // namespace gg
