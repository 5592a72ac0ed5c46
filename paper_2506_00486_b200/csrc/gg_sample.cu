// GG sampling for initialisation: x = alpha * sign * G^(1/beta), G ~ Gamma(1/beta, 1).
//
// If G ~ Gamma(1/beta, 1) then alpha G^(1/beta) with a fair sign has the density of Eq. 1
// (substitute y = (|x|/alpha)^beta).  G comes from the Marsaglia-Tsang method: shape a' = a
// (a >= 1) or a + 1 (a < 1), d = a' - 1/3, c = 1/sqrt(9 d); draw z ~ N(0,1), v = (1 + c z)^3,
// reject v <= 0, accept when ln u < z^2/2 + d (1 - v + ln v); G = d v, times u'^(1/a) if a < 1.
// Randomness is counter based (Philox4x32-10): attempt t of element i of tensor T uses the block
// at counter (i_lo, i_hi, t, T) under key (seed_lo, seed_hi); words 0,1 -> z by Box-Muller,
// word 2 -> u.  The block at t = 0xFFFFFFFF gives the sign (top bit of word 0) and u' (word 1).
// The work is fp64 transcendental throughput, not memory bandwidth.
#include <cuda_bf16.h>

#include "gg_internal.h"

namespace gg {
namespace {

constexpr int kThreads = 256;
constexpr uint32_t kMaxAttempts = 64;

struct Block4 { uint32_t w0, w1, w2, w3; };

// Philox4x32 with 10 rounds (Salmon et al., SC'11).
__device__ __forceinline__ Block4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                uint32_t k0, uint32_t k1)
{
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += W0;
        k1 += W1;
    }
    return Block4{c0, c1, c2, c3};
}

__device__ __forceinline__ double u01(uint32_t r) { return ((double)r + 0.5) * (1.0 / 4294967296.0); }

__device__ __forceinline__ float rcp_approx_f(float v)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

// Per-segment constants of the sampler.
struct GammaConst {
    double beta, alpha;
    double a;          // shape of the gamma variate, 1 / beta
    double d, c;       // Marsaglia-Tsang: d = a' - 1/3, c = 1 / sqrt(9 d)
    double ln_d;
};

__device__ __forceinline__ GammaConst gamma_const(double beta, double alpha)
{
    GammaConst k;
    k.beta = beta; k.alpha = alpha;
    k.a = 1.0 / beta;
    const double a1 = k.a >= 1.0 ? k.a : k.a + 1.0;
    k.d = a1 - 1.0 / 3.0;
    k.c = 1.0 / sqrt(9.0 * k.d);
    k.ln_d = log(k.d);
    return k;
}

// One attempt of the Marsaglia-Tsang method for element (i1, i0): true if it was accepted, with ln G in
// ln_g.  ln G = ln d + ln v, and ln v is needed by the acceptance test anyway.
__device__ __forceinline__ bool gamma_attempt(const GammaConst &k, uint32_t k0, uint32_t k1, uint32_t tensor, uint32_t i0,
                                              uint32_t i1, uint32_t t, double &ln_g)
{
    const Block4 r = philox4x32_10(i0, i1, t, tensor, k0, k1);
    // Box-Muller: cos(2 pi u) as cospi(2 u), whose argument reduction is exact
    const double z = sqrt(-2.0 * log(u01(r.w0))) * cospi(2.0 * u01(r.w1));
    const double w = 1.0 + k.c * z;
    if (w <= 0.0) return false;
    const double v = w * w * w;
    const double ln_v = log(v);
    // The acceptance test ln u < z^2/2 + d (1 - v + ln v) is decided from an fp32 logarithm whenever the
    // two sides are further apart than that logarithm can be wrong (1 ulp of logf and the rounding of u
    // to fp32 are below 3e-6 for ln u in (-22.2, 0)); only a tie within 1e-5 takes the fp64 logarithm.
    const double rhs = 0.5 * z * z + k.d * (1.0 - v + ln_v);
    const double u = u01(r.w2);
    const double ln_u32 = (double)logf((float)u);
    bool accept = ln_u32 + 1e-5 < rhs;
    if (!accept && !(ln_u32 - 1e-5 > rhs)) accept = log(u) < rhs;
    ln_g = k.ln_d + ln_v;
    return accept;
}

// The variate from an accepted ln G.  The power G^(1/beta) is taken in the log domain, so it costs one
// exp instead of a pow (and, for a < 1, one log instead of a second pow); the difference from pow is a
// few units of 1e-16 relative (times |ln x|), far below the storage types' rounding.
__device__ __forceinline__ double gg_from_gamma(const GammaConst &k, uint32_t k0, uint32_t k1, uint32_t tensor, uint32_t i0,
                                                uint32_t i1, double ln_g)
{
    const Block4 r = philox4x32_10(i0, i1, 0xFFFFFFFFu, tensor, k0, k1);
    if (k.a < 1.0) ln_g += log(u01(r.w1)) * k.beta;       // G u'^(1/a), 1/a = beta
    const double x = k.alpha * exp(ln_g * k.a);            // alpha G^(1/beta)
    return (r.w0 & 0x80000000u) ? -x : x;
}

// ---------------------------------------------------------------------------------------------------------
// bf16 output: attempt 0 in fp32 with running error bounds.
//
// A bf16 value keeps 8 significant bits, so the variate is needed to about 1e-3 relative: almost always an fp32
// evaluation of the same formulas lands in the same bf16 cell and on the same side of the acceptance test as the
// fp64 one.  The fp32 path therefore carries a bound on its own error (the documented bounds of logf, expf, cospif,
// with a factor of two to spare, and the roundings of the uniforms to 24 bits) and gives a result only when
//   * the acceptance test is decided with that bound to spare on either side, and
//   * the fp32 variate is further from the midpoint between two bf16 values than the bound (and is a normal number).
// Otherwise (about one element in a hundred) the element goes to the fp64 path from attempt 0, which is the
// definition.  What the fp32 path returns is therefore bit for bit what the fp64 path would.
enum : int { kFastAccept = 0, kFastReject = 1, kFastUnsure = 2 };

struct FastConst {
    float c, d, ln_d, a, beta, alpha;
    bool boost;        // a < 1: the variate is multiplied by u'^(1/a)
    bool usable;       // the constants are in a range where the bounds below hold
};

__device__ __forceinline__ FastConst fast_const(const GammaConst &k)
{
    FastConst f;
    f.c = (float)k.c; f.d = (float)k.d; f.ln_d = (float)k.ln_d; f.a = (float)k.a; f.beta = (float)k.beta; f.alpha = (float)k.alpha;
    f.boost = k.a < 1.0;
    // shapes between 0.1 and 8 and scales that are normal fp32 numbers: d <= 10, a <= 10, the exponent below stays
    // within the range where expf keeps its relative accuracy
    f.usable = k.beta >= 0.1 && k.beta <= 8.0 && k.alpha >= 1e-30 && k.alpha <= 1e30;
    return f;
}

// uniform (r + 1/2) 2^-32 to fp32: relative error below 1.2e-7 (the conversion of r and the addition)
__device__ __forceinline__ float u01f(uint32_t r) { return fmaf((float)r, 2.3283064365386963e-10f, 1.1641532182693481e-10f); }

// Attempt 0 of element (i1, i0) in fp32.  kFastAccept: *bits holds the bf16 pattern of the variate.
__device__ __forceinline__ int fast_attempt0(const FastConst &f, const Block4 &r, const Block4 &aux, uint16_t *bits)
{
    // ---- Box-Muller normal z with its error bound ez
    const float l0 = logf(u01f(r.w0));                       // <= 0; error 1.2e-7 (1 + |l0|)
    if (!(l0 < -1e-3f)) return kFastUnsure;                  // radius near zero: its relative error is unbounded here
    const float R = sqrtf(-2.0f * l0);
    // cos(2 pi u1) from the angle folded into the first quadrant in integers, so that the fp32 angle is exact to 1e-7 of pi/2
    const uint32_t quad = r.w1 >> 30;
    uint32_t frac = r.w1 & 0x3FFFFFFFu;
    if (quad & 1u) frac = 0x3FFFFFFFu - frac;
    float cs = cospif(fmaf((float)frac, 4.656612873077393e-10f, 2.3283064365386963e-10f));      // cos(pi/2 * (frac + 1/2) 2^-30)
    if ((quad + 1u) & 2u) cs = -cs;
    const float z = R * cs;
    const float ez = R * fmaf(6e-8f, rcp_approx_f(-l0), 5e-7f);
    // ---- Marsaglia-Tsang: w = 1 + c z, v = w^3, test ln u < z^2/2 + d (1 - v + ln v)
    const float w = fmaf(f.c, z, 1.0f);
    const float ew = fmaf(f.c, ez, 4e-7f);
    if (!(w > 8.0f * ew)) return kFastUnsure;                // w <= 0 rejects, but only the fp64 path may say so this close
    const float rw = rcp_approx_f(w);
    const float lw = logf(w);
    const float elw = fmaf(ew * 1.1f, rw, 1e-6f);            // (ew / w <= 1/8: the second-order term is within the 1.1)
    const float v = w * w * w;
    const float ev = v * fmaf(3.5f * ew, rw, 2e-7f);
    const float rhs = fmaf(0.5f * z, z, f.d * (1.0f - v + 3.0f * lw));
    // errors of z^2/2, of d (1 - v + 3 ln w), of the roundings of the sum (by its magnitude) and of ln u (3e-6)
    const float mag = fmaf(0.5f * z, z, f.d * (1.0f + v + 3.0f * fabsf(lw)));
    const float erhs = fmaf(fabsf(z), ez, fmaf(f.d, fmaf(3.0f, elw, ev), fmaf(2.4e-7f, mag, 5e-6f)));
    const float lu = logf(u01f(r.w2));
    if (lu - erhs > rhs) return kFastReject;
    if (!(lu + erhs < rhs)) return kFastUnsure;
    // ---- the variate alpha G^(1/beta), G = d v (times u'^(1/a) for a < 1), in the log domain
    float lg = fmaf(3.0f, lw, f.ln_d);
    float elg = fmaf(3.0f, elw, 3e-7f);
    if (f.boost) {
        const float lb = logf(u01f(aux.w1));
        lg = fmaf(f.beta, lb, lg);
        elg += f.beta * fmaf(2.5e-7f, -lb, 2.5e-7f);
    }
    elg = fmaf(1.2e-7f, fabsf(lg), elg);
    const float arg = lg * f.a;
    const float x = f.alpha * expf(arg);
    const float E = fmaf(f.a, elg, fmaf(1.2e-7f, fabsf(arg), 4e-7f));      // relative error bound of x
    const uint32_t xb = __float_as_uint(x);
    const uint32_t ex = xb >> 23;
    if (ex < 16u || ex > 250u) return kFastUnsure;                          // subnormal, zero, huge: the fp64 path rounds those
    const int low = (int)(xb & 0xFFFFu) - 0x8000;
    const float reach = fmaf(E, 33554432.0f, 2.0f);                         // the bound in fp32 ulps, twice over
    if (fabsf((float)low) <= reach) return kFastUnsure;
    *bits = (uint16_t)(((xb + 0x8000u) >> 16) | ((aux.w0 >> 16) & 0x8000u));
    return kFastAccept;
}

// fp64 -> bf16, round to nearest even in one step: truncate to fp32, fold everything that was
// dropped into the last fp32 bit (round to odd), then round the 16 spare bits away.
__device__ __forceinline__ uint16_t double_to_bf16(double x)
{
    float f = __double2float_rz(x);
    if ((double)f != x && f == f && fabsf(f) != INFINITY) f = __uint_as_float(__float_as_uint(f) | 1u);
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

template <typename T>
__device__ __forceinline__ void store_variate(T *out, double x)
{
    if constexpr (sizeof(T) == 4) *out = __double2float_rn(x);
    else *out = double_to_bf16(x);
}

// One CTA per tile.  Every element first gets attempt 0 (accepted with probability above 0.95 for every
// shape); the few rejected ones are queued in shared memory and finished afterwards, one per thread, so
// that a rejection does not make a whole warp walk the attempt loop again for one lane.
constexpr int kQueue = 2048;
template <typename T>
__global__ void __launch_bounds__(kThreads)
sample_kernel(const TileMap map, const double *beta, const double *alpha, uint32_t k0, uint32_t k1,
              uint32_t tensor_id0, uint32_t *max_attempts)
{
    __shared__ int queue[kQueue];
    __shared__ int n_queued;
    const int t = blockIdx.x;
    const int s = map.tile_seg[t];
    const int64_t len = map.seg_len[s];
    const int64_t off = (int64_t)(t - map.tile_prefix[s]) * kTile;
    const int n = (int)min((int64_t)kTile, len - off);
    T *out = reinterpret_cast<T *>(const_cast<void *>(map.seg_ptr[s])) + off;
    const GammaConst gk = gamma_const(beta[s], alpha[s]);
    const FastConst fk = fast_const(gk);
    const uint32_t tensor = tensor_id0 + (uint32_t)s;
    if (threadIdx.x == 0) n_queued = 0;
    __syncthreads();
    uint32_t worst = 0;
    // finishes element i from attempt t0 on
    auto finish = [&](int i, uint32_t t0) {
        const uint64_t index = (uint64_t)(off + i);
        const uint32_t i0 = (uint32_t)index, i1 = (uint32_t)(index >> 32);
        double ln_g = 0.0;
        uint32_t tt = t0;
        bool accepted = false;
        for (; tt < kMaxAttempts; ++tt) {
            if (gamma_attempt(gk, k0, k1, tensor, i0, i1, tt, ln_g)) { accepted = true; break; }
        }
        worst = max(worst, accepted ? tt + 1u : kMaxAttempts + 1u);
        store_variate<T>(out + i, accepted ? gg_from_gamma(gk, k0, k1, tensor, i0, i1, ln_g) : 0.0);
    };
    // (queue entries: the element in the low 16 bits, the attempt to start from above them)
    auto later = [&](int i, uint32_t t0) {
        const int q = atomicAdd(&n_queued, 1);
        if (q < kQueue) queue[q] = i | (int)(t0 << 16);
        else finish(i, t0);                            // (queue full: finish it here)
    };
    for (int i = threadIdx.x; i < n; i += kThreads) {
        const uint64_t index = (uint64_t)(off + i);
        const uint32_t i0 = (uint32_t)index, i1 = (uint32_t)(index >> 32);
        if constexpr (sizeof(T) == 2) {
            if (fk.usable) {
                const Block4 r = philox4x32_10(i0, i1, 0u, tensor, k0, k1);
                const Block4 aux = philox4x32_10(i0, i1, 0xFFFFFFFFu, tensor, k0, k1);
                uint16_t bits;
                const int verdict = fast_attempt0(fk, r, aux, &bits);
                if (verdict == kFastAccept) {
                    worst = max(worst, 1u);
                    out[i] = bits;
                } else {
                    later(i, verdict == kFastReject ? 1u : 0u);
                }
                continue;
            }
        }
        double ln_g;
        if (gamma_attempt(gk, k0, k1, tensor, i0, i1, 0u, ln_g)) {
            worst = max(worst, 1u);
            store_variate<T>(out + i, gg_from_gamma(gk, k0, k1, tensor, i0, i1, ln_g));
        } else {
            later(i, 1u);
        }
    }
    __syncthreads();
    const int nq = min(n_queued, kQueue);
    for (int q = threadIdx.x; q < nq; q += kThreads) finish(queue[q] & 0xFFFF, (uint32_t)queue[q] >> 16);
    if (max_attempts != nullptr) {
        worst = __reduce_max_sync(0xFFFFFFFFu, worst);
        if ((threadIdx.x & 31) == 0 && worst != 0) atomicMax(&max_attempts[s], worst);
    }
}

}  // namespace

cudaError_t launch_sample(const TileMap &map, gg_dtype dtype, const double *beta, const double *alpha,
                          uint64_t seed, uint32_t tensor_id0, uint32_t *max_attempts, cudaStream_t st)
{
    if (map.n_tiles <= 0) return cudaSuccess;
    const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    if (dtype == GG_F32)
        sample_kernel<float><<<map.n_tiles, kThreads, 0, st>>>(map, beta, alpha, k0, k1, tensor_id0, max_attempts);
    else
        sample_kernel<uint16_t><<<map.n_tiles, kThreads, 0, st>>>(map, beta, alpha, k0, k1, tensor_id0, max_attempts);
    return cudaGetLastError();
}

}  // namespace gg
