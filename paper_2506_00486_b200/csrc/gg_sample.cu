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
    for (int i = threadIdx.x; i < n; i += kThreads) {
        const uint64_t index = (uint64_t)(off + i);
        const uint32_t i0 = (uint32_t)index, i1 = (uint32_t)(index >> 32);
        double ln_g;
        if (gamma_attempt(gk, k0, k1, tensor, i0, i1, 0u, ln_g)) {
            worst = max(worst, 1u);
            store_variate<T>(out + i, gg_from_gamma(gk, k0, k1, tensor, i0, i1, ln_g));
        } else {
            const int q = atomicAdd(&n_queued, 1);
            if (q < kQueue) queue[q] = i;
            else finish(i, 1u);                        // (queue full: finish it here)
        }
    }
    __syncthreads();
    const int nq = min(n_queued, kQueue);
    for (int q = threadIdx.x; q < nq; q += kThreads) finish(queue[q], 1u);
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
