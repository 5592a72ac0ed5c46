// The channel-wise GG pass (one generalized Gaussian per column of a row-major matrix) for fp32 input.
//
// Same tiling as the bf16 kernels of gg_channels.cu with one column per lane: a strip of 32 columns is
// 128 contiguous bytes of every row, a warp reads one such row piece per load and walks down the rows.
// The fit and the penalty kernels are shared with the bf16 path (they work on the per-row-block partial
// sums).  Gradient: |x| = 2^(e-127) c (1 + r) with c = 1 + j/128 cut from the top seven mantissa bits, so
//     |g| = A_c[e] * B_c[j] * (1 + r)^b,    (1 + r)^b by a degree-4 binomial series in r < 2^-7,
// A and B per column (lane l reads word l of a table row: no bank conflicts), the series' coefficients in
// the lane's registers.  Exponents outside the 64 below the strip's largest magnitude, zero/subnormal,
// inf/nan, far binades and every element of a column with |b| > 2 read a NaN marker, which reaches the
// column's penalty partial of the current block of rows; that block's column then takes the exact fp64
// path.  Symbols are counted in a 4096-cell shared window; what falls outside is counted one by one.
#include <cuda_bf16.h>
#include <float.h>

#include "gg_fit_table.cuh"
#include "gg_device.cuh"
#include "gg_internal.h"

namespace gg {
namespace {

constexpr int kStrip = kChanStripF32;      // columns per strip = lanes
constexpr int kMomThreads = 256, kMomWarps = kMomThreads / 32;
constexpr int kU = 8;                      // rows in flight per thread and ring stage
constexpr int kTailThreads = 512, kTailWarps = kTailThreads / 32, kCtasPerSm = 2;
constexpr int kAWin = 64;                  // exponents covered by the A table (row kAWin: the marker)
constexpr int kSymWin = 4096;              // symbols counted in shared memory: [-2048, 2048) cut to [qmin, qmax]
constexpr int kTabFloats = (kAWin + 1) * 32 + 128 * 32;
static_assert(2 * kTabFloats == kChanTabFloats, "two fp32 strips take the table space of one bf16 strip");

__device__ __forceinline__ void moments_careful(uint32_t xb, double &s1, double &s2, uint32_t &bad)
{
    const uint32_t ax = xb & 0x7FFFFFFFu;
    if (ax < 0x7F800000u) {
        const double v = (double)__uint_as_float(ax);
        s1 += v;
        s2 += v * v;
    } else {
        bad += 1u;
    }
}

// One CTA per (strip, block of kChanMomRows rows): the lane sums its column over the rows of its warp
// (fp32 runs of eight rows, then fp64), the warps are added in a fixed order.
__global__ void __launch_bounds__(kMomThreads) chan_moments_f32_kernel(const ChanArgs a)
{
    __shared__ double red1[kMomWarps][kStrip], red2[kMomWarps][kStrip];
    __shared__ uint32_t redb[kMomWarps][kStrip];
    __shared__ float redmn[kMomWarps][kStrip], redmx[kMomWarps][kStrip];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t c = (int64_t)blockIdx.x * kStrip + lane;
    const int64_t r_begin = (int64_t)blockIdx.y * kChanMomRows, r_end = min(a.rows, r_begin + kChanMomRows);
    const bool ok = c < a.cols;
    const float *col = reinterpret_cast<const float *>(a.x) + c;
    double s1 = 0.0, s2 = 0.0;
    uint32_t bad = 0;
    float mn = INFINITY, mx = -INFINITY;
    const int64_t stride = (int64_t)kMomWarps * a.ld;
    const float *p = col + (r_begin + warp) * a.ld;
    for (int64_t r = r_begin + warp; r < r_end; r += (int64_t)kMomWarps * kU, p += kU * stride) {
        const int nvalid = (int)min((int64_t)kU, (r_end - r + kMomWarps - 1) / kMomWarps);
        float x[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) x[u] = (ok && u < nvalid) ? __ldg(p + u * stride) : 0.0f;
        float m1 = 0.0f, m2 = 0.0f;
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            m1 += fabsf(x[u]);
            m2 = fmaf(x[u], x[u], m2);
            if (u < nvalid) {                      // (padding must not enter the extremes)
                mn = fminf(mn, x[u]);              // fminf / fmaxf return the non-NaN operand
                mx = fmaxf(mx, x[u]);
            }
        }
        if (run_sums_exact_enough(m1, m2)) {
            s1 += (double)m1;
            s2 += (double)m2;
        } else {     // an inf or nan (left out of the sums and counted), or squares outside the fp32 range
#pragma unroll
            for (int u = 0; u < kU; ++u)
                if (u < nvalid) moments_careful(__float_as_uint(x[u]), s1, s2, bad);
        }
    }
    red1[warp][lane] = s1; red2[warp][lane] = s2; redb[warp][lane] = bad; redmn[warp][lane] = mn; redmx[warp][lane] = mx;
    __syncthreads();
    if (threadIdx.x < kStrip && (int64_t)blockIdx.x * kStrip + threadIdx.x < a.cols) {
        double r1 = 0.0, r2 = 0.0;
        uint32_t rb = 0;
        float rmn = INFINITY, rmx = -INFINITY;
        for (int w = 0; w < kMomWarps; ++w) {     // fixed order
            r1 += red1[w][threadIdx.x]; r2 += red2[w][threadIdx.x]; rb += redb[w][threadIdx.x];
            rmn = fminf(rmn, redmn[w][threadIdx.x]); rmx = fmaxf(rmx, redmx[w][threadIdx.x]);
        }
        const int64_t o = (int64_t)blockIdx.y * a.cols + (int64_t)blockIdx.x * kStrip + threadIdx.x;
        a.s1[o] = r1; a.s2[o] = r2; a.bad[o] = rb; a.xmin[o] = rmn; a.xmax[o] = rmx;
    }
}

// One CTA per strip: the gradient tables of its 32 columns, A [i][lane] then B [j][lane], and the exponent
// field of the first A row.
__global__ void __launch_bounds__(256) chan_tables_f32_kernel(const ChanArgs a)
{
    __shared__ double colL[kStrip], colb[kStrip], lg[128];
    __shared__ int e_top;
    const int tid = threadIdx.x, strip = blockIdx.x;
    const uint32_t flip = a.lambda < 0.0 ? 0x80000000u : 0u;
    if (tid == 0) e_top = 0;
    if (tid < 128) lg[tid] = log2(1.0 + (double)tid * (1.0 / 128.0));
    __syncthreads();
    if (tid < kStrip) {
        const int64_t c = (int64_t)strip * kStrip + tid;
        const bool ok = c < a.cols;
        colL[tid] = ok ? a.L[c] : __longlong_as_double(0x7FF8000000000000ll);
        colb[tid] = ok ? a.b[c] : 0.0;
        if (ok) atomicMax(&e_top, (int)(__float_as_uint(a.amax[c]) >> 23));
    }
    __syncthreads();
    const int e_lo = max(1, min(e_top, 254) - (kAWin - 1));
    if (tid == 0) a.tab_elo[strip] = e_lo;
    float *ta = a.tab + (int64_t)strip * kTabFloats, *tb = ta + (kAWin + 1) * 32;
    for (int idx = tid; idx < (kAWin + 1) * 32; idx += blockDim.x) {
        const int l = idx & 31, i = idx >> 5;
        const double L = colL[l], b = colb[l];
        float v = 0.0f;                                  // a column without gradient: zero everywhere
        if (L == L) {
            // One fp32 factor serves an exponent if its product with B and the series stays in the normal range
            // (|L + b (e-127)| <= 100) and the series applies (|b| <= 2); the rest, and the last row, hold the marker.
            const int e = e_lo + i;
            const double e0 = L + b * (double)(e - 127);
            v = __int_as_float(0x7FC00000);
            if (i < kAWin && e <= 254 && fabs(e0) <= 100.0 && fabs(b) <= 2.0)
                v = __uint_as_float(__float_as_uint((float)exp2_short(e0)) ^ flip);
        }
        ta[idx] = v;
    }
    for (int idx = tid; idx < 128 * 32; idx += blockDim.x) {
        const int l = idx & 31, j = idx >> 5;
        tb[idx] = (colL[l] == colL[l]) ? (float)exp2_short(colb[l] * lg[j]) : 1.0f;
    }
}

// ------------------------------------------------------------------------------------ second kernel

struct ConstF32 {           // warp-uniform constants that only the cold paths need
    float inv;
    int32_t wlo, whi, qmin, qmax;
    uint32_t flip;
    unsigned long long *hist;
};

struct SmemF32 {
    uint32_t ring[2][kU][kTailThreads];   // per-thread slots of the rows in flight: two blocks of kU rows
    float a1[kAWin + 1][32];              // [e - e_lo][lane]; row kAWin: the marker
    float bt[128][32];                    // [j][lane]
    uint32_t cnt[kSymWin + 2];            // cell 0 and cell whi - wlo + 1: sentinels of the two tails
    double red[kTailWarps][kStrip];
    double colL[kStrip], colb[kStrip];
    uint32_t clampc[2];
    ConstF32 cc;
};

struct LaneF32 {
    uint32_t a_addr, b_addr;         // shared-memory addresses of this lane's word in row 0 of the tables
    uint32_t e_lo;
    uint32_t cnt_off;                // cell of a value = bits(floor(t) + magic) * 4 + cnt_off (mod 2^32)
    float inv, t_lo, t_hi, near;     // quantiser scale; clamp of t; a smaller |t| is inside the window for sure
    float c1, c2, c3, c4;            // binomial coefficients of (1 + r)^b for the lane's column
};

// Exact gradient magnitude (with lambda's sign through `flip`) of |x| given as fp32 bits.
__device__ __noinline__ float grad_exact_f32(uint32_t ax, double L, double b, uint32_t flip)
{
    const float v = __uint_as_float(ax);
    if (!(L == L) || v == 0.0f) return 0.0f;
    const float g = (float)exp2(L + b * log2((double)v));
    return __uint_as_float(__float_as_uint(g) ^ flip);
}

__device__ __noinline__ double pen_exact_f32(uint32_t ax, double L, double b)
{
    const double v = (double)__uint_as_float(ax);
    if (!(L == L) || v == 0.0) return 0.0;
    return v * exp2(L + b * log2(v));
}

// Quantises one value and counts its symbol: the shared window when in reach, else global memory.
__device__ __noinline__ void count_slow_f32(float x, SmemF32 *sm)
{
    const float t = __fmul_rn(x, sm->cc.inv);
    if (t == t) {                                  // NaN is skipped
        int q = __float2int_rd(t);                 // floor, saturating
        if (q < sm->cc.qmin) { q = sm->cc.qmin; atomicAdd(&sm->clampc[0], 1u); }
        else if (q > sm->cc.qmax) { q = sm->cc.qmax; atomicAdd(&sm->clampc[1], 1u); }
        if (q >= sm->cc.wlo && q < sm->cc.whi) atomicAdd(&sm->cnt[q - sm->cc.wlo + 1], 1u);
        else atomicAdd(&sm->cc.hist[q - sm->cc.qmin], 1ull);
    }
}

// One element (fp32 bits).  Branch free; see the head of the file.
template <bool GRAD, bool HIST>
__device__ __forceinline__ float elem_f32(uint32_t xb, bool counted, const LaneF32 &ln, float &mp, float &anyc)
{
    const float x = __uint_as_float(xb);
    float g = 0.0f;
    if constexpr (GRAD) {
        const uint32_t ax = xb & 0x7FFFFFFFu;
        const uint32_t i = min((ax >> 23) - ln.e_lo, (uint32_t)kAWin);       // below the window wraps around to the marker too
        const float av = lds_f32(ln.a_addr + i * 128u);
        const float bj = lds_f32(ln.b_addr + ((ax >> 16) & 127u) * 128u);
        const float c = __uint_as_float((ax & 0x007F0000u) | 0x3F800000u);      // 1 + j/128
        const float m = __uint_as_float((ax & 0x007FFFFFu) | 0x3F800000u);
        const float r = (m - c) * rcp_approx(c);                                 // m = c (1 + r), m - c exact
        const float t = r * fmaf(r, fmaf(r, fmaf(r, ln.c4, ln.c3), ln.c2), ln.c1);   // (1 + r)^b - 1
        float ga = av * fmaf(bj, t, bj);
        ga = ax == 0u ? 0.0f : ga;                                               // g(0) = 0 for every shape
        mp = fmaf(fabsf(x), fabsf(ga), mp);
        g = __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));           // the table carries lambda's sign
    }
    if constexpr (HIST) {
        if (counted) {
            const float t = __fmul_rn(x, ln.inv);
            anyc = fmaxf(anyc, fabsf(t));      // (a nan is ignored here and lands on a sentinel: nan is not counted)
            const float tc = fminf(fmaxf(t, ln.t_lo), ln.t_hi);
            const uint32_t fb = __float_as_uint(__fadd_rd(tc, __uint_as_float(kMagicBits)));
            red_inc(fb * 4u + ln.cnt_off);
        }
    }
    return g;
}

template <typename TG>
__device__ __forceinline__ void store_g(TG *p, float g, bool accumulate)
{
    if constexpr (sizeof(TG) == 4) {
        *p = accumulate ? *p + g : g;
    } else {
        if (accumulate) g += __uint_as_float((uint32_t)*p << 16);
        *p = __bfloat16_as_ushort(__float2bfloat16_rn(g));
    }
}

// kU rows of the lane's column: row u is word_of(u) (fp32 bits; rows past nvalid and a missing column read as
// zero and are not counted).  Gradients wait in registers until the exact path has run.
template <typename TG, bool GRAD, bool HIST, typename WordOf>
__device__ __forceinline__ void block_f32(WordOf word_of, TG *gp, int64_t sg, int nvalid, bool ok, bool accumulate, int lane,
                                          const LaneF32 &ln, SmemF32 &sm, double &pen)
{
    float g[kU];
    float mp = 0.0f, anyc = 0.0f;
#pragma unroll
    for (int u = 0; u < kU; ++u) g[u] = elem_f32<GRAD, HIST>(word_of(u), ok && u < nvalid, ln, mp, anyc);
    if constexpr (GRAD) {
        if (mp <= FLT_MAX) {
            pen += (double)mp;
        } else {     // a marker, or a product beyond the fp32 range: this column's rows again, exactly
            const double L = sm.colL[lane], b = sm.colb[lane];
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const uint32_t xb = word_of(u), ax = xb & 0x7FFFFFFFu;
                pen += pen_exact_f32(ax, L, b);            // (rows past the end read as zero: no term)
                const float av = lds_f32(ln.a_addr + min((ax >> 23) - ln.e_lo, (uint32_t)kAWin) * 128u);
                if (av != av && ax != 0u)
                    g[u] = __uint_as_float(__float_as_uint(grad_exact_f32(ax, L, b, sm.cc.flip)) ^ (xb & 0x80000000u));
            }
        }
    }
    if constexpr (HIST) {
        if (anyc >= ln.near) {      // some symbol may have missed the window (it was counted in a sentinel)
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const float x = __uint_as_float(word_of(u));
                const float t = __fmul_rn(x, ln.inv);
                if (ok && u < nvalid && !(t >= (float)sm.cc.wlo && t < (float)sm.cc.whi)) count_slow_f32(x, &sm);
            }
        }
    }
    if constexpr (GRAD) {
        if (gp != nullptr && ok) {
#pragma unroll
            for (int u = 0; u < kU; ++u)
                if (u < nvalid) store_g<TG>(gp + u * sg, g[u], accumulate);
        }
    }
}

template <typename TG, bool GRAD, bool HIST>
__global__ void __launch_bounds__(kTailThreads, kCtasPerSm) chan_tail_f32_kernel(const ChanArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemF32 &sm = *reinterpret_cast<SmemF32 *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_strips = (int)((a.cols + kStrip - 1) / kStrip);
    const int n_items = n_strips * a.n_slices;
    const int32_t wlo = (int32_t)max((int64_t)-kSymWin / 2, (int64_t)a.qmin);
    const int32_t whi = (int32_t)max((int64_t)wlo, min((int64_t)kSymWin / 2, (int64_t)a.qmax + 1));
    const float inv = (float)(1.0 / (double)a.step);
    if (tid == 0) {
        sm.cc.inv = inv; sm.cc.wlo = wlo; sm.cc.whi = whi; sm.cc.qmin = a.qmin; sm.cc.qmax = a.qmax;
        sm.cc.flip = a.lambda < 0.0 ? 0x80000000u : 0u;
        sm.cc.hist = reinterpret_cast<unsigned long long *>(a.hist);
    }
    LaneF32 ln;
    ln.a_addr = (uint32_t)__cvta_generic_to_shared(&sm.a1[0][lane]);
    ln.b_addr = (uint32_t)__cvta_generic_to_shared(&sm.bt[0][lane]);
    ln.e_lo = 1u;
    ln.inv = inv;
    ln.t_lo = (float)wlo - 0.5f;
    ln.t_hi = (float)whi;
    ln.near = (wlo < 0 && whi > 0) ? (float)min(-wlo, whi) : 0.0f;
    ln.cnt_off = (uint32_t)__cvta_generic_to_shared(sm.cnt) - (kMagicBits + (uint32_t)(wlo - 1)) * 4u;
    ln.c1 = ln.c2 = ln.c3 = ln.c4 = 0.0f;
    if constexpr (HIST) {
        for (int i = tid; i < kSymWin + 2; i += kTailThreads) sm.cnt[i] = 0u;
        if (tid < 2) sm.clampc[tid] = 0u;
    }
    const bool accumulate = a.accumulate != 0;
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(&sm.ring[0][0][tid]);
    constexpr uint32_t kRowBytes = kTailThreads * 4u;
    int cur_strip = -1;
    __syncthreads();

    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int strip = item % n_strips, slice = item / n_strips;
        // slices are cut at multiples of the rows one pass of the CTA covers, so that only the last one is ragged
        constexpr int64_t kPass = (int64_t)kTailWarps * kU;
        const int64_t n_pass = (a.rows + kPass - 1) / kPass;
        const int64_t r_begin = n_pass * slice / a.n_slices * kPass;
        const int64_t r_end = min(a.rows, n_pass * (slice + 1) / a.n_slices * kPass);
        const int64_t c = (int64_t)strip * kStrip + lane;
        const bool ok = c < a.cols;

        if (GRAD && strip != cur_strip) {
            cur_strip = strip;
            __syncthreads();
            const uint4 *src = reinterpret_cast<const uint4 *>(a.tab + (int64_t)strip * kTabFloats);
            uint4 *dst = reinterpret_cast<uint4 *>(&sm.a1[0][0]);      // a1 and bt are contiguous
            for (int i = tid; i < kTabFloats / 4; i += kTailThreads) dst[i] = __ldg(src + i);
            if (tid < kStrip) {
                const int64_t cc = (int64_t)strip * kStrip + tid;
                const bool okc = cc < a.cols;
                sm.colL[tid] = okc ? a.L[cc] : __longlong_as_double(0x7FF8000000000000ll);
                sm.colb[tid] = okc ? a.b[cc] : 0.0;
            }
            ln.e_lo = (uint32_t)__ldg(a.tab_elo + strip);
            const float bf = ok ? (float)a.b[c] : 0.0f;
            ln.c1 = bf;
            ln.c2 = ln.c1 * (bf - 1.0f) * 0.5f;
            ln.c3 = ln.c2 * (bf - 2.0f) * (1.0f / 3.0f);
            ln.c4 = ln.c3 * (bf - 3.0f) * 0.25f;
            __syncthreads();
        }

        double pen = 0.0;
        const int64_t r0 = r_begin + warp;
        int n_mine = r0 < r_end ? (int)((r_end - r0 + kTailWarps - 1) / kTailWarps) : 0;      // rows of this warp
        const int64_t sin = (int64_t)kTailWarps * a.ld, sg = (int64_t)kTailWarps * a.grad_ld;
        const float *p = reinterpret_cast<const float *>(a.x) + c + r0 * a.ld;
        TG *gp = GRAD && a.grad != nullptr ? reinterpret_cast<TG *>(a.grad) + c + r0 * a.grad_ld : nullptr;
        if (ok) {
            // whole blocks: the thread stages its words of the next block in its own ring slots with asynchronous
            // copies while it works on the current one (one commit group per block)
            const int n_blocks = n_mine / kU;
            auto stage = [&](const float *src, uint32_t dst) {
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
                block_f32<TG, GRAD, HIST>([&](int u) {
                    uint32_t w;
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(cur + (uint32_t)u * kRowBytes));
                    return w;
                }, gp, sg, kU, true, accumulate, lane, ln, sm, pen);
                p += kU * sin;
                if (gp != nullptr) gp += kU * sg;
            }
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            n_mine -= n_blocks * kU;
        }
        for (; n_mine > 0; n_mine -= kU, p += kU * sin, gp += gp != nullptr ? kU * sg : 0) {
            uint32_t w[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) w[u] = (ok && u < n_mine) ? __float_as_uint(__ldg(p + u * sin)) : 0u;
            block_f32<TG, GRAD, HIST>([&](int u) { return w[u]; }, gp, sg, min(n_mine, kU), ok, accumulate, lane, ln, sm, pen);
        }

        if constexpr (GRAD) {
            sm.red[warp][lane] = pen;
            __syncthreads();
            if (tid < kStrip) {
                const int64_t cc = (int64_t)strip * kStrip + tid;
                if (cc < a.cols) {
                    double ps = 0.0;
                    for (int wv = 0; wv < kTailWarps; ++wv) ps += sm.red[wv][tid];     // fixed order
                    a.pen[(int64_t)slice * a.cols + cc] = ps;
                }
            }
            __syncthreads();
        }
    }

    if constexpr (HIST) {
        __syncthreads();
        unsigned long long *hist = reinterpret_cast<unsigned long long *>(a.hist);
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
cudaError_t launch_typed(const ChanArgs &a, int grid, cudaStream_t st)
{
    void (*kern)(const ChanArgs) = nullptr;
    if (a.do_grad && a.do_hist) kern = chan_tail_f32_kernel<TG, true, true>;
    else if (a.do_grad) kern = chan_tail_f32_kernel<TG, true, false>;
    else kern = chan_tail_f32_kernel<TG, false, true>;
    // more than 48 KB of dynamic shared memory needs the opt-in (per function and device)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(SmemF32));
    if (e != cudaSuccess) return e;
    kern<<<grid, kTailThreads, sizeof(SmemF32), st>>>(a);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_chan_moments_f32(const ChanArgs &a, cudaStream_t st)
{
    if (a.rows <= 0 || a.cols <= 0) return cudaSuccess;
    const dim3 grid((unsigned)((a.cols + kStrip - 1) / kStrip), (unsigned)a.n_mom_blocks);
    chan_moments_f32_kernel<<<grid, kMomThreads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_chan_tail_f32(gg_dtype grad_dtype, const ChanArgs &a, int sm_count, cudaStream_t st)
{
    if (a.rows <= 0 || a.cols <= 0 || (!a.do_grad && !a.do_hist)) return cudaSuccess;
    const int64_t n_strips = (a.cols + kStrip - 1) / kStrip;
    const int grid = (int)min(n_strips * a.n_slices, (int64_t)sm_count * kCtasPerSm);
    if (a.do_grad) {
        chan_tables_f32_kernel<<<(unsigned)n_strips, 256, 0, st>>>(a);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (a.grad != nullptr && grad_dtype == GG_BF16) return launch_typed<uint16_t>(a, grid, st);
    return launch_typed<float>(a, grid, st);
}

}  // namespace gg
