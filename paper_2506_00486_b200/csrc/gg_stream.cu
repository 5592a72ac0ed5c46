// The streaming kernel of the GG pass: one CTA per tile of one segment.  Depending on the
// template flags a sweep accumulates the moments (sum |x|, sum x^2), writes the penalty gradient
// and the penalty partial, and counts quantised symbols into a shared-memory histogram window.
//
// Memory behaviour: each tile is read once with 128-bit loads (several in flight per thread),
// the gradient is written once with 128-bit stores; everything else stays on chip until the
// per-tile partials and the non-empty histogram bins are flushed.
#include <cuda_bf16.h>
#include <float.h>

#include "gg_device.cuh"
#include "gg_internal.h"

namespace gg {
namespace {

constexpr int kThreads = kStreamThreads;
constexpr int kWarps = kThreads / 32;
constexpr int kUnroll = 4;          // 128-bit loads in flight per thread
constexpr int kATab = 280;          // exponent table: unbiased exponents -150 .. 129
constexpr int kBTab = 128;          // mantissa table: top 7 mantissa bits

// ---------------------------------------------------------------------------- element types
template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kVec = 4;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[4])
    {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ float load(const float *p) { return __ldg(p); }
    static __device__ __forceinline__ float to_float(float v) { return v; }
    static __device__ __forceinline__ float from_float(float v) { return v; }
};
template <> struct Elem<uint16_t> {   // bf16 as raw bits: widening is a 16-bit shift, exact
    static constexpr int kVec = 8;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&f)[8])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ float load(const uint16_t *p)
    {
        return __uint_as_float((uint32_t)__ldg(p) << 16);
    }
    static __device__ __forceinline__ float to_float(uint16_t v) { return __uint_as_float((uint32_t)v << 16); }
    static __device__ __forceinline__ uint16_t from_float(float v)
    {
        return __bfloat16_as_ushort(__float2bfloat16_rn(v));
    }
};

// Stores KV consecutive gradient values at g (16-byte aligned), optionally adding to what is there.
template <typename TG, int KV>
__device__ __forceinline__ void store_vec(TG *g, const float (&v)[KV], bool accumulate)
{
    if constexpr (sizeof(TG) == 4) {
        float4 *p = reinterpret_cast<float4 *>(g);
#pragma unroll
        for (int i = 0; i < KV / 4; ++i) {
            float4 o = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            if (accumulate) {
                const float4 old = p[i];
                o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
            }
            p[i] = o;
        }
    } else {
        uint32_t w[KV / 2];
        uint32_t *p = reinterpret_cast<uint32_t *>(g);
#pragma unroll
        for (int i = 0; i < KV / 2; ++i) {
            float lo = v[2 * i], hi = v[2 * i + 1];
            if (accumulate) {
                const uint32_t old = p[i];
                lo += __uint_as_float(old << 16);
                hi += __uint_as_float(old & 0xFFFF0000u);
            }
            w[i] = (uint32_t)Elem<uint16_t>::from_float(lo) | ((uint32_t)Elem<uint16_t>::from_float(hi) << 16);
        }
        if constexpr (KV == 8) {
            *reinterpret_cast<uint4 *>(g) = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
            *reinterpret_cast<uint2 *>(g) = make_uint2(w[0], w[1]);
        }
    }
}

// ---------------------------------------------------------------------------- gradient math
//
// g = sign(x) * 2^(L + b log2|x|),  L = log2(lambda beta) - beta log2(alpha),  b = beta - 1.
//
// Fast path (|b| <= 2, normal finite x).  Write |x| = 2^e * m, m in [1,2), and let j be the top 7
// bits of m's fraction.  With invc_j = fl32(1/(1 + j/128)) and r = fma(m, invc_j, -1) the identity
// m = (1 + r)/invc_j holds up to one rounding of r (|r| < 2^-7), so
//     |g| = [2^(L + b e)] * [invc_j^-b] * (1 + r)^b.
// The first bracket is a per-exponent table A[e] = (A1, A2) with A1*A2 the value and A2 a power of
// two that keeps A1 in the normal range; the second a per-j table B[j]; both are built in fp64 by
// the CTA for its segment.  (1 + r)^b is the degree-4 binomial series (next term < 2e-10).
// Rounding: A1, B, fma(B, t, B) and the product A1*p each round once; the multiplication by A2 is
// exact unless the result is subnormal or overflows, where it is the single final rounding.
// Total <= 2 ulp.  Everything else (zero, subnormal, inf, nan inputs; |b| > 2) takes the fp64 path.
__device__ __noinline__ float grad_slow(float x, double L, double b)
{
    const float ax = fabsf(x);
    if (ax == 0.0f) return 0.0f;
    const double g = exp2(L + b * log2((double)ax));
    return (float)g;     // round-to-nearest conversion: overflow -> inf, subnormals rounded once
}

struct GradConst {
    float c1, c2, c3, c4;   // binomial coefficients of (1 + r)^b
    double L, b;
    uint32_t sign_flip;     // 0x80000000 if lambda < 0
    int mode;               // 0: zeros, 1: table path, 2: fp64 path
};

__device__ __forceinline__ float grad_elem(float x, const GradConst &k, const float2 *A, const float2 *B)
{
    const uint32_t bits = __float_as_uint(x);
    const uint32_t ax = bits & 0x7FFFFFFFu;
    float g;
    if (k.mode == 1) {
        const uint32_t ef = ax >> 23;
        if (ef - 1u < 254u) {   // normal and finite
            const float2 a = A[ef + 23];
            const float2 bj = B[(ax >> 16) & 127u];
            const float m = __uint_as_float((ax & 0x007FFFFFu) | 0x3F800000u);
            const float r = fmaf(m, bj.x, -1.0f);
            const float t = r * fmaf(r, fmaf(r, fmaf(r, k.c4, k.c3), k.c2), k.c1);
            const float p = fmaf(bj.y, t, bj.y);
            g = (a.x * p) * a.y;
        } else {
            g = grad_slow(x, k.L, k.b);
        }
    } else if (k.mode == 2) {
        g = grad_slow(x, k.L, k.b);
    } else {
        return 0.0f;
    }
    return __uint_as_float(__float_as_uint(g) | ((bits & 0x80000000u) ^ k.sign_flip));
}

// ---------------------------------------------------------------------------- per-thread state
struct Acc {
    double s1 = 0.0, s2 = 0.0, pen = 0.0;
    uint32_t bad = 0;
    float xmin = INFINITY, xmax = -INFINITY;
};

struct HistConst {
    float inv;
    int32_t qmin, qmax;
    unsigned long long *row;   // this segment's histogram, bin 0 = symbol qmin
};

__device__ __forceinline__ void hist_elem(float x, const HistConst &h, uint32_t *win, uint32_t *clampc)
{
    const float t = __fmul_rn(x, h.inv);
    if (t == t) {                       // NaN is skipped
        int q = __float2int_rd(t);      // floor, saturating
        if (q < h.qmin) { q = h.qmin; atomicAdd(&clampc[0], 1u); }
        else if (q > h.qmax) { q = h.qmax; atomicAdd(&clampc[1], 1u); }
        const uint32_t w = (uint32_t)(q + kWindow / 2);
        if (w < (uint32_t)kWindow) atomicAdd(&win[w], 1u);
        else atomicAdd(&h.row[q - h.qmin], 1ull);
    }
}

template <int FLAGS, int KV>
__device__ __forceinline__ void process(const float (&x)[KV], float (&g)[KV], Acc &acc,
                                        const GradConst &gc, const HistConst &hc, const float2 *A,
                                        const float2 *B, uint32_t *win, uint32_t *clampc)
{
    float m1 = 0.0f, m2 = 0.0f, mp = 0.0f;
#pragma unroll
    for (int e = 0; e < KV; ++e) {
        const float xe = x[e];
        const float ax = fabsf(xe);
        if constexpr (FLAGS & kMoments) {
            const bool fin = ax <= FLT_MAX;          // false for inf and nan
            const float af = fin ? ax : 0.0f;
            m1 += af;
            m2 = fmaf(af, af, m2);
            acc.bad += fin ? 0u : 1u;
            acc.xmin = fminf(acc.xmin, xe);      // fminf / fmaxf return the non-NaN operand
            acc.xmax = fmaxf(acc.xmax, xe);
        }
        if constexpr (FLAGS & kGrad) {
            const float ge = grad_elem(xe, gc, A, B);
            g[e] = ge;
            mp = fmaf(ax, fabsf(ge), mp);
        }
        if constexpr (FLAGS & kHist) hist_elem(xe, hc, win, clampc);
    }
    // short fp32 runs, then fp64: the fp32 part adds at most KV roundings of 2^-24 each
    if constexpr (FLAGS & kMoments) {
        if (run_sums_exact_enough(m1, m2)) {
            acc.s1 += (double)m1;
            acc.s2 += (double)m2;
        } else {     // a square or a sum outside the fp32 range: this run again in fp64
            for (int e = 0; e < KV; ++e) {
                const double ax = (double)fabsf(x[e]);
                if (ax <= (double)FLT_MAX) { acc.s1 += ax; acc.s2 += ax * ax; }
            }
        }
    }
    if constexpr (FLAGS & kGrad) {
        if (mp <= FLT_MAX) {
            acc.pen += (double)mp;
        } else {   // a product or a gradient left the fp32 range (or is nan): redo this run in fp64
            double dp = 0.0;
            for (int e = 0; e < KV; ++e) {
                const double ax = (double)fabsf(x[e]);
                if (ax != 0.0 && gc.mode != 0) dp += ax * exp2(gc.L + gc.b * log2(ax));
            }
            acc.pen += dp;
        }
    }
}

// ---------------------------------------------------------------------------- the kernel
template <typename TIn, typename TG, int FLAGS>
__global__ void __launch_bounds__(kThreads) stream_kernel(const StreamArgs a)
{
    constexpr int KV = Elem<TIn>::kVec;
    constexpr bool MOM = (FLAGS & kMoments) != 0, GRAD = (FLAGS & kGrad) != 0, HIST = (FLAGS & kHist) != 0;

    __shared__ float2 shA[GRAD ? kATab : 1];
    __shared__ float2 shB[GRAD ? kBTab : 1];
    __shared__ uint32_t shWin[HIST ? kWindow : 1];
    __shared__ uint32_t shClamp[2];
    __shared__ double shL;
    __shared__ double shRed[3][kWarps];
    __shared__ uint32_t shBad[kWarps];
    __shared__ float shMin[kWarps], shMax[kWarps];

    const int tid = threadIdx.x;
    const int t = blockIdx.x;
    const int s = a.map.tile_seg[t];
    const int64_t len = a.map.seg_len[s];
    const int64_t off = (int64_t)(t - a.map.tile_prefix[s]) * kTile;
    const int n = (int)min((int64_t)kTile, len - off);
    const TIn *x = reinterpret_cast<const TIn *>(a.map.seg_ptr[s]) + off;
    TG *gout = nullptr;
    if constexpr (GRAD) {
        if (a.map.grad_ptr != nullptr) gout = reinterpret_cast<TG *>(a.map.grad_ptr[s]) + off;
    }

    GradConst gc{};
    HistConst hc{};
    int hid = 0;

    if constexpr (GRAD) {
        const double beta = a.beta[s], alpha = a.alpha[s];
        const double lam = a.mean_reduction ? a.lambda / (double)len : a.lambda;
        gc.b = beta - 1.0;
        gc.sign_flip = lam < 0.0 ? 0x80000000u : 0u;
        if (!(beta > 0.0) || !(alpha > 0.0) || lam == 0.0 || !(lam == lam)) gc.mode = 0;
        else gc.mode = fabs(gc.b) <= 2.0 ? 1 : 2;
        if (gc.mode != 0) {
            if (tid == 0) shL = log2(fabs(lam) * beta) - beta * log2(alpha);
            __syncthreads();
            gc.L = shL;
        }
        if (gc.mode == 1) {
            for (int k = tid; k < kATab; k += kThreads) {
                const double e0 = gc.L + gc.b * (double)(k - 150);
                double ip = rint(e0);
                const double f = exp2(e0 - ip);
                ip = fmin(fmax(ip, -400.0), 400.0);
                const int ii = (int)ip;
                const int i1 = max(-100, min(100, ii));
                const int i2 = max(-126, min(126, ii - i1));
                shA[k] = make_float2((float)ldexp(f, i1), __int_as_float((i2 + 127) << 23));
            }
            for (int j = tid; j < kBTab; j += kThreads) {
                const float invc = __frcp_rn(1.0f + (float)j * (1.0f / 128.0f));
                shB[j] = make_float2(invc, (float)exp2(-gc.b * log2((double)invc)));
            }
            const float bf = (float)gc.b;
            gc.c1 = bf;
            gc.c2 = gc.c1 * (bf - 1.0f) * 0.5f;
            gc.c3 = gc.c2 * (bf - 2.0f) * (1.0f / 3.0f);
            gc.c4 = gc.c3 * (bf - 3.0f) * 0.25f;
        }
    }
    if constexpr (HIST) {
        for (int i = tid; i < kWindow; i += kThreads) shWin[i] = 0u;
        if (tid < 2) shClamp[tid] = 0u;
        hid = a.map.hist_id ? a.map.hist_id[s] : s;
        hc.inv = (float)(1.0 / (double)a.step[s]);
        hc.qmin = a.qmin;
        hc.qmax = a.qmax;
        hc.row = reinterpret_cast<unsigned long long *>(a.hist) +
                 (int64_t)hid * ((int64_t)a.qmax - (int64_t)a.qmin + 1);
    }
    if constexpr (GRAD || HIST) __syncthreads();

    // Split the tile into a scalar head (up to the first 16-byte boundary of x), a body of
    // 128-bit vectors, and a scalar tail.  If the gradient's address is not 16-byte aligned at
    // the same element, the whole tile takes the scalar route.
    int head = (int)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / sizeof(TIn));
    head = min(head, n);
    if (gout != nullptr && (reinterpret_cast<uintptr_t>(gout + head) & 15u) != 0) head = n;
    // (the body starts a 512-byte block of the gradient, or of x when there is none)
    else head = (int)aligned_head(head, n, reinterpret_cast<uintptr_t>(x), reinterpret_cast<uintptr_t>(gout), (unsigned)sizeof(TIn),
                                  (unsigned)sizeof(TG), 512u);
    const int nvec = (n - head) / KV;
    const int tail0 = head + nvec * KV;
    const bool accumulate = GRAD && a.accumulate != 0;

    Acc acc;
    for (int i = tid; i < head + (n - tail0); i += kThreads) {
        const int idx = i < head ? i : tail0 + (i - head);
        const float xe[1] = {Elem<TIn>::load(x + idx)};
        float ge[1] = {0.0f};
        process<FLAGS, 1>(xe, ge, acc, gc, hc, shA, shB, shWin, shClamp);
        if constexpr (GRAD) {
            if (gout != nullptr) {
                float v = ge[0];
                if (accumulate) v += Elem<TG>::to_float(gout[idx]);
                gout[idx] = Elem<TG>::from_float(v);
            }
        }
    }

    const uint4 *xv = reinterpret_cast<const uint4 *>(x + head);
    for (int v0 = tid; v0 < nvec; v0 += kThreads * kUnroll) {
        uint4 raw[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int v = v0 + u * kThreads;
            if (v < nvec) raw[u] = __ldg(xv + v);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int v = v0 + u * kThreads;
            if (v < nvec) {
                float xe[KV], ge[KV];
                Elem<TIn>::unpack(raw[u], xe);
                process<FLAGS, KV>(xe, ge, acc, gc, hc, shA, shB, shWin, shClamp);
                if constexpr (GRAD) {
                    if (gout != nullptr) store_vec<TG, KV>(gout + head + (int64_t)v * KV, ge, accumulate);
                }
            }
        }
    }

    // Block reduction in a fixed order: butterfly inside each warp, then warps 0..7 in sequence.
    const int lane = tid & 31, warp = tid >> 5;
    if constexpr (MOM) {
        const double w1 = warp_sum(acc.s1), w2 = warp_sum(acc.s2);
        const uint32_t wb = __reduce_add_sync(0xFFFFFFFFu, acc.bad);
        float wmin = acc.xmin, wmax = acc.xmax;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            wmin = fminf(wmin, __shfl_xor_sync(0xFFFFFFFFu, wmin, o));
            wmax = fmaxf(wmax, __shfl_xor_sync(0xFFFFFFFFu, wmax, o));
        }
        if (lane == 0) {
            shRed[0][warp] = w1; shRed[1][warp] = w2; shBad[warp] = wb;
            shMin[warp] = wmin; shMax[warp] = wmax;
        }
    }
    if constexpr (GRAD) {
        const double wp = warp_sum(acc.pen);
        if (lane == 0) shRed[2][warp] = wp;
    }
    __syncthreads();
    if (tid == 0) {
        if constexpr (MOM) {
            double r1 = 0.0, r2 = 0.0;
            uint32_t rb = 0;
            float rmin = INFINITY, rmax = -INFINITY;
            for (int w = 0; w < kWarps; ++w) {
                r1 += shRed[0][w]; r2 += shRed[1][w]; rb += shBad[w];
                rmin = fminf(rmin, shMin[w]); rmax = fmaxf(rmax, shMax[w]);
            }
            a.part.s1[t] = r1; a.part.s2[t] = r2; a.part.bad[t] = rb;
            a.part.xmin[t] = rmin; a.part.xmax[t] = rmax;
        }
        if constexpr (GRAD) {
            double rp = 0.0;
            for (int w = 0; w < kWarps; ++w) rp += shRed[2][w];
            a.part.pen[t] = gc.sign_flip ? -rp : rp;   // the penalty carries lambda's sign
        }
    }
    if constexpr (HIST) {
        // (the __syncthreads above also orders every shared-memory atomic before this flush)
        for (int i = tid; i < kWindow; i += kThreads) {
            const uint32_t c = shWin[i];
            if (c != 0u) atomicAdd(&hc.row[(i - kWindow / 2) - hc.qmin], (unsigned long long)c);
        }
        if (tid < 2 && shClamp[tid] != 0u) {
            if (a.clamped != nullptr)
                atomicAdd(reinterpret_cast<unsigned long long *>(a.clamped) + 2 * hid + tid,
                          (unsigned long long)shClamp[tid]);
        }
    }
}

// ---------------------------------------------------------------------------- bf16 moments
// The first sweep over bf16 data reads 2 bytes per element, so at HBM speed an SM has about ten
// issue slots per element.  This kernel spends about five: the widening and the two sums per
// element and min/max on packed bf16 pairs; a vector whose fp32 sum of squares comes out inf or nan
// (it holds an inf or a nan, or values whose squares leave the fp32 range) is redone element by
// element in fp64.
__device__ __forceinline__ void moments_careful(uint32_t h, double &m1, double &m2, uint32_t &bad)
{
    const uint32_t mag = h & 0x7FFFu;
    const double ax = (double)__uint_as_float(mag << 16);
    if (mag < 0x7F80u) { m1 += ax; m2 = fma(ax, ax, m2); }     // (fp64: a square above 3.4e38 must not become inf)
    else bad += 1u;
}

__global__ void __launch_bounds__(kThreads) moments_bf16_kernel(const StreamArgs a)
{
    __shared__ double shRed[2][kWarps];
    __shared__ uint32_t shBad[kWarps];
    __shared__ float shMin[kWarps], shMax[kWarps];
    const int tid = threadIdx.x;
    const int t = blockIdx.x;
    const int s = a.map.tile_seg[t];
    const int64_t len = a.map.seg_len[s];
    const int64_t off = (int64_t)(t - a.map.tile_prefix[s]) * kTile;
    const int n = (int)min((int64_t)kTile, len - off);
    const uint16_t *x = reinterpret_cast<const uint16_t *>(a.map.seg_ptr[s]) + off;
    int head = (int)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / 2u);
    head = (int)aligned_head(head, n, reinterpret_cast<uintptr_t>(x), 0ull, 2u, 0u, 512u);      // (the body starts a 512-byte block of x)
    const int nvec = (n - head) / 8;
    const int tail0 = head + nvec * 8;

    double s1 = 0.0, s2 = 0.0;
    uint32_t bad = 0;
    float xmin = INFINITY, xmax = -INFINITY;
    for (int i = tid; i < head + (n - tail0); i += kThreads) {
        const int idx = i < head ? i : tail0 + (i - head);
        const uint32_t h = (uint32_t)__ldg(x + idx);
        moments_careful(h, s1, s2, bad);
        xmin = fminf(xmin, __uint_as_float(h << 16));
        xmax = fmaxf(xmax, __uint_as_float(h << 16));
    }
    __nv_bfloat162 mn2 = __floats2bfloat162_rn(INFINITY, INFINITY), mx2 = __floats2bfloat162_rn(-INFINITY, -INFINITY);
    const uint4 *xv = reinterpret_cast<const uint4 *>(x + head);
    for (int v0 = tid; v0 < nvec; v0 += kThreads * kUnroll) {
        uint4 raw[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int v = v0 + u * kThreads;
            if (v < nvec) raw[u] = __ldg(xv + v);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int v = v0 + u * kThreads;
            if (v < nvec) {
                const uint32_t w[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
                float m1 = 0.0f, m2 = 0.0f;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
                    m1 += fabsf(lo);
                    m1 += fabsf(hi);
                    m2 = fmaf(lo, lo, m2);
                    m2 = fmaf(hi, hi, m2);
                    const __nv_bfloat162 p = *reinterpret_cast<const __nv_bfloat162 *>(&w[i]);
                    mn2 = __hmin2(mn2, p);      // return the non-NaN operand, like fminf
                    mx2 = __hmax2(mx2, p);
                }
                if (!run_sums_exact_enough(m1, m2)) {
                    // an inf or nan in this vector (to be left out of the sums), or squares outside the fp32
                    // range: the vector again, element by element in fp64
                    for (int i = 0; i < 4; ++i) {
                        moments_careful(w[i] & 0xFFFFu, s1, s2, bad);
                        moments_careful(w[i] >> 16, s1, s2, bad);
                    }
                } else {
                    s1 += (double)m1;
                    s2 += (double)m2;
                }
            }
        }
    }
    xmin = fminf(xmin, fminf(__low2float(mn2), __high2float(mn2)));
    xmax = fmaxf(xmax, fmaxf(__low2float(mx2), __high2float(mx2)));

    const int lane = tid & 31, warp = tid >> 5;
    const double w1 = warp_sum(s1), w2 = warp_sum(s2);
    const uint32_t wb = __reduce_add_sync(0xFFFFFFFFu, bad);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        xmin = fminf(xmin, __shfl_xor_sync(0xFFFFFFFFu, xmin, o));
        xmax = fmaxf(xmax, __shfl_xor_sync(0xFFFFFFFFu, xmax, o));
    }
    if (lane == 0) { shRed[0][warp] = w1; shRed[1][warp] = w2; shBad[warp] = wb; shMin[warp] = xmin; shMax[warp] = xmax; }
    __syncthreads();
    if (tid == 0) {
        double r1 = 0.0, r2 = 0.0;
        uint32_t rb = 0;
        float rmin = INFINITY, rmax = -INFINITY;
        for (int w = 0; w < kWarps; ++w) {
            r1 += shRed[0][w]; r2 += shRed[1][w]; rb += shBad[w];
            rmin = fminf(rmin, shMin[w]); rmax = fmaxf(rmax, shMax[w]);
        }
        a.part.s1[t] = r1; a.part.s2[t] = r2; a.part.bad[t] = rb;
        a.part.xmin[t] = rmin; a.part.xmax[t] = rmax;
    }
}

// The same sums by persistent CTAs (two of 512 threads per SM), each walking one contiguous range of
// tiles: inside a segment that range is one run of elements, streamed as 128-bit vectors through a
// per-thread ring of asynchronous copies (four vectors in flight per thread and no registers held by
// them), so that the block reduction, the partial-sum stores and the address set-up are paid once per
// run instead of once per 32 KB tile.  A run's sums go to the slot of its first tile, zeros to the
// slots of its other tiles.
constexpr int kSweepThreads = 512, kSweepWarps = kSweepThreads / 32, kSweepCtasPerSm = 2, kSweepDepth = 4;

__device__ __forceinline__ void moments_vec(const uint4 &raw, double &s1, double &s2, uint32_t &bad, __nv_bfloat162 &mn2,
                                            __nv_bfloat162 &mx2)
{
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    float m1 = 0.0f, m2 = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
        m1 += fabsf(lo);
        m1 += fabsf(hi);
        m2 = fmaf(lo, lo, m2);
        m2 = fmaf(hi, hi, m2);
        const __nv_bfloat162 p = *reinterpret_cast<const __nv_bfloat162 *>(&w[i]);
        mn2 = __hmin2(mn2, p);      // return the non-NaN operand, like fminf
        mx2 = __hmax2(mx2, p);
    }
    if (run_sums_exact_enough(m1, m2)) {
        s1 += (double)m1;
        s2 += (double)m2;
    } else {
        // an inf or nan in this vector (to be left out of the sums), or squares outside the fp32 range: the
        // vector again, element by element in fp64
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            moments_careful(w[i] & 0xFFFFu, s1, s2, bad);
            moments_careful(w[i] >> 16, s1, s2, bad);
        }
    }
}

__global__ void __launch_bounds__(kSweepThreads, kSweepCtasPerSm) moments_bf16_sweep_kernel(const StreamArgs a)
{
    __shared__ uint4 stage[kSweepDepth][kSweepThreads];
    __shared__ double shRed[2][kSweepWarps];
    __shared__ uint32_t shBad[kSweepWarps];
    __shared__ float shMin[kSweepWarps], shMax[kSweepWarps];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t nt = a.map.n_tiles;
    const int t_begin = (int)(nt * blockIdx.x / gridDim.x);
    const int t_end = (int)(nt * (blockIdx.x + 1) / gridDim.x);
    const uint32_t slot0 = (uint32_t)__cvta_generic_to_shared(&stage[0][tid]);
    constexpr uint32_t kStageBytes = sizeof(uint4) * kSweepThreads;

    // this CTA's share of the memory to clear for the sweep that follows (plain stores, a few per thread)
    if (a.zero_ptr != nullptr) {
        const int64_t z0 = a.zero_vecs * blockIdx.x / gridDim.x, z1 = a.zero_vecs * (blockIdx.x + 1) / gridDim.x;
        for (int64_t z = z0 + tid; z < z1; z += kSweepThreads) a.zero_ptr[z] = make_uint4(0u, 0u, 0u, 0u);
    }

    for (int t = t_begin; t < t_end;) {
        // ---- one run: the tiles of this CTA's range that lie in segment s
        const int s = a.map.tile_seg[t];
        const int64_t len = a.map.seg_len[s];
        const int t_first = a.map.tile_prefix[s];
        const int t_stop = min(t_end, a.map.tile_prefix[s + 1]);
        const int64_t off = (int64_t)(t - t_first) * kTile;
        const int64_t n = min(len, (int64_t)(t_stop - t_first) * kTile) - off;
        const uint16_t *x = reinterpret_cast<const uint16_t *>(a.map.seg_ptr[s]) + off;
        int64_t head = (int64_t)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / 2u);
        head = aligned_head(head, n, reinterpret_cast<uintptr_t>(x), 0ull, 2u, 0u, 512u);      // (the body starts a 512-byte block of x)
        const int nv = (int)((n - head) / 8);      // (a CTA's run never exceeds device memory / grid size elements)
        const int64_t tail0 = head + (int64_t)nv * 8;

        double s1 = 0.0, s2 = 0.0;
        uint32_t bad = 0;
        float xmin = INFINITY, xmax = -INFINITY;
        for (int64_t i = tid; i < head + (n - tail0); i += kSweepThreads) {
            const int64_t idx = i < head ? i : tail0 + (i - head);
            if (!GG_IN_BOUNDS(idx, n)) continue;
            const uint32_t h = (uint32_t)__ldg(x + idx);
            moments_careful(h, s1, s2, bad);
            xmin = fminf(xmin, __uint_as_float(h << 16));
            xmax = fmaxf(xmax, __uint_as_float(h << 16));
        }
        __nv_bfloat162 mn2 = __floats2bfloat162_rn(INFINITY, INFINITY), mx2 = __floats2bfloat162_rn(-INFINITY, -INFINITY);
        // Each thread owns slot [d][tid] of every stage d: it fills them with asynchronous 16-byte copies (one
        // commit group per vector, empty past the end so that the group count stays in step) and reads a slot
        // back once the group that filled it has landed.
        const uint4 *xv = reinterpret_cast<const uint4 *>(x + head) + tid;
#pragma unroll
        for (int d = 0; d < kSweepDepth - 1; ++d) {
            if (tid + d * kSweepThreads < nv && GG_IN_BOUNDS(head + (int64_t)(tid + d * kSweepThreads) * 8 + 7, n))
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot0 + d * kStageBytes), "l"(xv + d * kSweepThreads) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        for (int v = tid; v < nv; v += kSweepDepth * kSweepThreads) {
#pragma unroll
            for (int d = 0; d < kSweepDepth; ++d) {
                const int vd = v + d * kSweepThreads;
                if (vd < nv) {
                    // fill the slot emptied by the previous vector (stage d - 1, cyclically)
                    if (vd + (kSweepDepth - 1) * kSweepThreads < nv && GG_IN_BOUNDS(head + (int64_t)(vd + (kSweepDepth - 1) * kSweepThreads) * 8 + 7, n))
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot0 + ((d + kSweepDepth - 1) % kSweepDepth) * kStageBytes),
                                     "l"(xv + (d + kSweepDepth - 1) * kSweepThreads) : "memory");
                    asm volatile("cp.async.commit_group;" ::: "memory");
                    asm volatile("cp.async.wait_group %0;" ::"n"(kSweepDepth - 1) : "memory");
                    uint4 r0;
                    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r0.x), "=r"(r0.y), "=r"(r0.z), "=r"(r0.w) : "r"(slot0 + d * kStageBytes) : "memory");
                    moments_vec(r0, s1, s2, bad, mn2, mx2);
                }
            }
            xv += kSweepDepth * kSweepThreads;
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        xmin = fminf(xmin, fminf(__low2float(mn2), __high2float(mn2)));
        xmax = fmaxf(xmax, fmaxf(__low2float(mx2), __high2float(mx2)));

        // ---- block reduction in a fixed order: butterfly inside each warp, then the warps in sequence
        const double w1 = warp_sum(s1), w2 = warp_sum(s2);
        const uint32_t wb = __reduce_add_sync(0xFFFFFFFFu, bad);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            xmin = fminf(xmin, __shfl_xor_sync(0xFFFFFFFFu, xmin, o));
            xmax = fmaxf(xmax, __shfl_xor_sync(0xFFFFFFFFu, xmax, o));
        }
        if (lane == 0) { shRed[0][warp] = w1; shRed[1][warp] = w2; shBad[warp] = wb; shMin[warp] = xmin; shMax[warp] = xmax; }
        __syncthreads();
        for (int tz = t + 1 + tid; tz < t_stop; tz += kSweepThreads) {
            a.part.s1[tz] = 0.0; a.part.s2[tz] = 0.0; a.part.bad[tz] = 0u;
            a.part.xmin[tz] = INFINITY; a.part.xmax[tz] = -INFINITY;
        }
        if (tid == 0) {
            double r1 = 0.0, r2 = 0.0;
            uint32_t rb = 0;
            float rmin = INFINITY, rmax = -INFINITY;
            for (int w = 0; w < kSweepWarps; ++w) {
                r1 += shRed[0][w]; r2 += shRed[1][w]; rb += shBad[w];
                rmin = fminf(rmin, shMin[w]); rmax = fmaxf(rmax, shMax[w]);
            }
            a.part.s1[t] = r1; a.part.s2[t] = r2; a.part.bad[t] = rb;
            a.part.xmin[t] = rmin; a.part.xmax[t] = rmax;
        }
        __syncthreads();
        t = t_stop;
    }
}

template <typename TIn, typename TG>
cudaError_t launch_typed(int flags, const StreamArgs &a, cudaStream_t st)
{
    const dim3 grid((unsigned)a.map.n_tiles), block(kThreads);
    switch (flags) {
    case kMoments: stream_kernel<TIn, TG, kMoments><<<grid, block, 0, st>>>(a); break;
    case kGrad: stream_kernel<TIn, TG, kGrad><<<grid, block, 0, st>>>(a); break;
    case kHist: stream_kernel<TIn, TG, kHist><<<grid, block, 0, st>>>(a); break;
    case kGrad | kHist: stream_kernel<TIn, TG, kGrad | kHist><<<grid, block, 0, st>>>(a); break;
    case kMoments | kGrad: stream_kernel<TIn, TG, kMoments | kGrad><<<grid, block, 0, st>>>(a); break;
    case kMoments | kHist: stream_kernel<TIn, TG, kMoments | kHist><<<grid, block, 0, st>>>(a); break;
    case kMoments | kGrad | kHist:
        stream_kernel<TIn, TG, kMoments | kGrad | kHist><<<grid, block, 0, st>>>(a);
        break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_stream(int flags, gg_dtype in_dtype, gg_dtype grad_dtype, bool has_grad_out,
                          const StreamArgs &a, cudaStream_t st)
{
    if (a.map.n_tiles <= 0) return cudaSuccess;
    if (in_dtype == GG_BF16 && flags == kMoments) {
        moments_bf16_kernel<<<(unsigned)a.map.n_tiles, kThreads, 0, st>>>(a);
        return cudaGetLastError();
    }
    // without a gradient output the gradient type does not matter: use one instantiation
    const bool g16 = has_grad_out && grad_dtype == GG_BF16;
    if (in_dtype == GG_F32)
        return g16 ? launch_typed<float, uint16_t>(flags, a, st) : launch_typed<float, float>(flags, a, st);
    return g16 ? launch_typed<uint16_t, uint16_t>(flags, a, st) : launch_typed<uint16_t, float>(flags, a, st);
}

cudaError_t launch_moments_bf16_sweep(const StreamArgs &a, int sm_count, cudaStream_t st)
{
    if (a.map.n_tiles <= 0) return cudaSuccess;
    const int grid = (int)min((int64_t)a.map.n_tiles, (int64_t)sm_count * kSweepCtasPerSm);
    moments_bf16_sweep_kernel<<<grid, kSweepThreads, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace gg
