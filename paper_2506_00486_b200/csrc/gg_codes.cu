// Code-length side of the rate model: the Exponential-Golomb rate of Eq. 6-7 from a symbol histogram,
// its elementwise gradient, and the elementwise update of gradient constrained training
// (Algorithm 2).  All three are streaming or O(bins) kernels; none is a contraction.
#include <cuda_bf16.h>

#include "gg_internal.h"

namespace gg {
namespace {

constexpr int kThreads = 256;
constexpr unsigned kFull = 0xFFFFFFFFu;

// Eq. 6: signed symbol -> unsigned symbol.
__device__ __forceinline__ uint32_t map_unsigned(int32_t q)
{
    return q < 0 ? (uint32_t)(-2 * (int64_t)q) : (q == 0 ? 0u : (uint32_t)(2 * (int64_t)q - 1));
}

// Length of the k-th order Exponential-Golomb code of m: 2 floor(log2(m + 2^k)) - k + 1.
__device__ __forceinline__ int eg_length(uint32_t m, int k)
{
    const unsigned long long v = (unsigned long long)m + (1ull << k);
    return 2 * (63 - __clzll((long long)v)) - k + 1;
}

// One CTA per histogram: sum of count * length and sum of counts in 64-bit integers (exact, so the
// order of the additions does not matter), then the mean.
__global__ void __launch_bounds__(kThreads) eg_rate_kernel(const uint64_t *hist, int32_t n_bins, int32_t qmin, int32_t k,
                                                           double *eg_bits)
{
    __shared__ unsigned long long shBits[kThreads / 32], shTot[kThreads / 32];
    const uint64_t *row = hist + (int64_t)blockIdx.x * n_bins;
    unsigned long long bits = 0, tot = 0;
    for (int b = threadIdx.x; b < n_bins; b += kThreads) {
        const unsigned long long c = row[b];
        if (c != 0) {
            bits += c * (unsigned long long)eg_length(map_unsigned(qmin + b), k);
            tot += c;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        bits += __shfl_xor_sync(kFull, bits, o);
        tot += __shfl_xor_sync(kFull, tot, o);
    }
    if ((threadIdx.x & 31) == 0) { shBits[threadIdx.x >> 5] = bits; shTot[threadIdx.x >> 5] = tot; }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long rb = 0, rt = 0;
        for (int w = 0; w < kThreads / 32; ++w) { rb += shBits[w]; rt += shTot[w]; }
        eg_bits[blockIdx.x] = rt ? (double)rb / (double)rt : 0.0;
    }
}

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<uint16_t>(uint16_t v) { return __uint_as_float((uint32_t)v << 16); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ uint16_t from_f32<uint16_t>(float v) { return __bfloat16_as_ushort(__float2bfloat16_rn(v)); }

// The unsigned symbol of x plus 2^k, as the quantiser defines it (fp32 product, floor, clamp), or 0
// when x is zero or nan (no gradient there).
__device__ __forceinline__ uint32_t eg_denominator(float x, float inv, int32_t qmin, int32_t qmax, int k)
{
    const float t = __fmul_rn(x, inv);
    if (!(t == t) || x == 0.0f) return 0u;
    const int q = max(qmin, min(qmax, __float2int_rd(t)));      // floor, saturating, then the clamp
    return map_unsigned(q) + (1u << k);
}

// Four consecutive elements at p (aligned to four elements) or one element, as fp32.
template <typename T> struct Vec4;
template <> struct Vec4<float> {
    static __device__ __forceinline__ void load(const float *p, float (&v)[4])
    {
        const float4 t = __ldcs(reinterpret_cast<const float4 *>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&v)[4])
    {
        __stcs(reinterpret_cast<float4 *>(p), make_float4(v[0], v[1], v[2], v[3]));
    }
};
template <> struct Vec4<uint16_t> {
    static __device__ __forceinline__ void load(const uint16_t *p, float (&v)[4])
    {
        const uint2 t = __ldcs(reinterpret_cast<const uint2 *>(p));
        v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xFFFF0000u);
        v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xFFFF0000u);
    }
    static __device__ __forceinline__ void store(uint16_t *p, const float (&v)[4])
    {
        uint2 t;
        t.x = (uint32_t)from_f32<uint16_t>(v[0]) | ((uint32_t)from_f32<uint16_t>(v[1]) << 16);
        t.y = (uint32_t)from_f32<uint16_t>(v[2]) | ((uint32_t)from_f32<uint16_t>(v[3]) << 16);
        __stcs(reinterpret_cast<uint2 *>(p), t);
    }
};

template <typename T>
__device__ __forceinline__ bool aligned4(const T *p) { return (reinterpret_cast<uintptr_t>(p) & (4 * sizeof(T) - 1)) == 0; }

// Gradient of lambda * R (Eq. 7) for every element: one CTA per tile, four elements per thread and
// trip when the tile's addresses allow vector accesses.
//     g = lambda * 4 inv / (N ln 2) * sign(x) / (Map(q) + 2^k)
// The per-segment factor is formed in fp64 and rounded once; the division is one fp32 rounding.
template <typename TIn, typename TG>
__global__ void __launch_bounds__(kThreads) eg_grad_kernel(const TileMap map, const float *step, int32_t qmin, int32_t qmax,
                                                           int32_t k, double lambda, int accumulate)
{
    const int t = blockIdx.x;
    const int s = map.tile_seg[t];
    const int64_t len = map.seg_len[s];
    const int64_t off = (int64_t)(t - map.tile_prefix[s]) * kTile;
    const int n = (int)min((int64_t)kTile, len - off);
    const TIn *x = reinterpret_cast<const TIn *>(map.seg_ptr[s]) + off;
    TG *g = reinterpret_cast<TG *>(map.grad_ptr[s]) + off;
    const float inv = (float)(1.0 / (double)step[s]);
    const float c = (float)(lambda * 4.0 * (double)inv / ((double)len * 0.6931471805599453094));
    auto one = [&](float xv, float old) {
        const uint32_t den = eg_denominator(xv, inv, qmin, qmax, k);
        float v = 0.0f;
        if (den != 0u) {
            v = __fdiv_rn(c, (float)den);       // (den is exact in fp32 up to 2^24: symbols of any 16-bit alphabet)
            if (xv < 0.0f) v = -v;
        }
        return accumulate ? v + old : v;
    };
    const int nvec = (aligned4(x) && aligned4(g)) ? n / 4 : 0;
    for (int v = threadIdx.x; v < nvec; v += kThreads) {
        float xv[4], gv[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        Vec4<TIn>::load(x + 4 * v, xv);
        if (accumulate) Vec4<TG>::load(g + 4 * v, gv);
#pragma unroll
        for (int i = 0; i < 4; ++i) gv[i] = one(xv[i], gv[i]);
        Vec4<TG>::store(g + 4 * v, gv);
    }
    for (int i = 4 * nvec + threadIdx.x; i < n; i += kThreads)
        g[i] = from_f32<TG>(one(to_f32<TIn>(x[i]), accumulate ? to_f32<TG>(g[i]) : 0.0f));
}

// Algorithm 2, the three elementwise lines, one CTA per tile.  The curvature estimate
// 1 - g / (ghat_prev + eps) cancels, so that quotient and what follows are fp64 (one fp64 division
// per element fits under the time the five streams of four bytes take); the reciprocal of dR/dg's
// integer denominator is an fp32 reciprocal refined by one fp64 Newton step.  Storage fp32.
template <typename TIn>
__global__ void __launch_bounds__(kThreads) gct_step_kernel(const TileMap map, void *const *w_ptr, const float *step,
                                                            int32_t qmin, int32_t qmax, int32_t k, double eta, double lambda,
                                                            double eps, int apply_h)
{
    const int t = blockIdx.x;
    const int s = map.tile_seg[t];
    const int64_t len = map.seg_len[s];
    const int64_t off = (int64_t)(t - map.tile_prefix[s]) * kTile;
    const int n = (int)min((int64_t)kTile, len - off);
    const TIn *g = reinterpret_cast<const TIn *>(map.seg_ptr[s]) + off;
    float *ghat = reinterpret_cast<float *>(map.grad_ptr[s]) + off;
    float *w = reinterpret_cast<float *>(w_ptr[s]) + off;
    const float inv = (float)(1.0 / (double)step[s]);
    const double c = lambda * 4.0 * (double)inv / ((double)len * 0.6931471805599453094);
    const double inv_eta = 1.0 / eta;
    auto one = [&](float gf, float &gh_io, float &w_io) {
        const double gd = (double)gf;
        double gh = gd;
        if (apply_h) {
            const uint32_t den = eg_denominator(gf, inv, qmin, qmax, k);
            if (den != 0u) {
                // 1 / den: an fp32 reciprocal and one Newton step in fp64 (error ~1e-14), cheaper than a division
                const double r0 = (double)__frcp_rn((float)den);
                const double rcp = r0 * fma(-(double)den, r0, 2.0);
                const double rate_term = (gf < 0.0f ? -c : c) * rcp;     // lambda dR/dg
                const double h = inv_eta - inv_eta * gd / ((double)gh_io + eps);
                gh = fma(rate_term, h, gd);
            }
        }
        gh_io = (float)gh;
        w_io = (float)fma(-eta, gh, (double)w_io);
    };
    const int nvec = (aligned4(g) && aligned4(ghat) && aligned4(w)) ? n / 4 : 0;
    for (int v = threadIdx.x; v < nvec; v += kThreads) {
        float gv[4], hv[4], wv[4];
        Vec4<TIn>::load(g + 4 * v, gv);
        Vec4<float>::load(ghat + 4 * v, hv);
        Vec4<float>::load(w + 4 * v, wv);
#pragma unroll
        for (int i = 0; i < 4; ++i) one(gv[i], hv[i], wv[i]);
        Vec4<float>::store(ghat + 4 * v, hv);
        Vec4<float>::store(w + 4 * v, wv);
    }
    for (int i = 4 * nvec + threadIdx.x; i < n; i += kThreads) one(to_f32<TIn>(g[i]), ghat[i], w[i]);
}

}  // namespace

namespace {
__global__ void eg_penalty_kernel(const double *eg_bits, const int32_t *hist_id, double lambda, double *penalty, int32_t n_seg)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s < n_seg) penalty[s] = lambda * eg_bits[hist_id[s]];
}
}  // namespace

cudaError_t launch_eg_penalty(const double *eg_bits, const int32_t *hist_id, double lambda, double *penalty, int32_t n_seg,
                              cudaStream_t st)
{
    if (n_seg <= 0) return cudaSuccess;
    eg_penalty_kernel<<<(n_seg + 255) / 256, 256, 0, st>>>(eg_bits, hist_id, lambda, penalty, n_seg);
    return cudaGetLastError();
}

cudaError_t launch_eg_rate(const uint64_t *hist, int32_t n_hist, int32_t n_bins, int32_t qmin, int32_t k, double *eg_bits,
                           cudaStream_t st)
{
    if (n_hist <= 0) return cudaSuccess;
    eg_rate_kernel<<<n_hist, kThreads, 0, st>>>(hist, n_bins, qmin, k, eg_bits);
    return cudaGetLastError();
}

cudaError_t launch_eg_grad(const TileMap &map, gg_dtype in_dtype, gg_dtype grad_dtype, const float *step, int32_t qmin,
                           int32_t qmax, int32_t k, double lambda, int accumulate, cudaStream_t st)
{
    if (map.n_tiles <= 0) return cudaSuccess;
    const dim3 grid((unsigned)map.n_tiles), block(kThreads);
    if (in_dtype == GG_F32 && grad_dtype == GG_F32) eg_grad_kernel<float, float><<<grid, block, 0, st>>>(map, step, qmin, qmax, k, lambda, accumulate);
    else if (in_dtype == GG_F32) eg_grad_kernel<float, uint16_t><<<grid, block, 0, st>>>(map, step, qmin, qmax, k, lambda, accumulate);
    else if (grad_dtype == GG_F32) eg_grad_kernel<uint16_t, float><<<grid, block, 0, st>>>(map, step, qmin, qmax, k, lambda, accumulate);
    else eg_grad_kernel<uint16_t, uint16_t><<<grid, block, 0, st>>>(map, step, qmin, qmax, k, lambda, accumulate);
    return cudaGetLastError();
}

cudaError_t launch_gct_step(const TileMap &map, void *const *w_ptr, gg_dtype g_dtype, const float *step, int32_t qmin,
                            int32_t qmax, int32_t k, double eta, double lambda, double eps, int apply_h, cudaStream_t st)
{
    if (map.n_tiles <= 0) return cudaSuccess;
    const dim3 grid((unsigned)map.n_tiles), block(kThreads);
    if (g_dtype == GG_F32) gct_step_kernel<float><<<grid, block, 0, st>>>(map, w_ptr, step, qmin, qmax, k, eta, lambda, eps, apply_h);
    else gct_step_kernel<uint16_t><<<grid, block, 0, st>>>(map, w_ptr, step, qmin, qmax, k, eta, lambda, eps, apply_h);
    return cudaGetLastError();
}

}  // namespace gg
