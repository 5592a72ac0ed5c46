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

__device__ __forceinline__ double gg_variate(double beta, double alpha, uint32_t k0, uint32_t k1,
                                             uint32_t tensor, uint64_t index, uint32_t &attempts)
{
    const uint32_t i0 = (uint32_t)index, i1 = (uint32_t)(index >> 32);
    const double a = 1.0 / beta;
    const double a1 = a >= 1.0 ? a : a + 1.0;
    const double d = a1 - 1.0 / 3.0;
    const double c = 1.0 / sqrt(9.0 * d);
    double G = 0.0;
    bool accepted = false;
    uint32_t t = 0;
    for (; t < kMaxAttempts; ++t) {
        const Block4 r = philox4x32_10(i0, i1, t, tensor, k0, k1);
        const double z = sqrt(-2.0 * log(u01(r.w0))) * cos(6.283185307179586476925286766559 * u01(r.w1));
        const double w = 1.0 + c * z;
        if (w <= 0.0) continue;
        const double v = w * w * w;
        if (log(u01(r.w2)) < 0.5 * z * z + d * (1.0 - v + log(v))) {
            G = d * v;
            accepted = true;
            break;
        }
    }
    attempts = accepted ? t + 1u : kMaxAttempts + 1u;
    if (!accepted) return 0.0;
    const Block4 r = philox4x32_10(i0, i1, 0xFFFFFFFFu, tensor, k0, k1);
    if (a < 1.0) G *= pow(u01(r.w1), 1.0 / a);
    const double x = alpha * pow(G, 1.0 / beta);
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
__global__ void __launch_bounds__(kThreads)
sample_kernel(const TileMap map, const double *beta, const double *alpha, uint32_t k0, uint32_t k1,
              uint32_t tensor_id0, uint32_t *max_attempts)
{
    const int t = blockIdx.x;
    const int s = map.tile_seg[t];
    const int64_t len = map.seg_len[s];
    const int64_t off = (int64_t)(t - map.tile_prefix[s]) * kTile;
    const int n = (int)min((int64_t)kTile, len - off);
    T *out = reinterpret_cast<T *>(const_cast<void *>(map.seg_ptr[s])) + off;
    const double b = beta[s], al = alpha[s];
    uint32_t worst = 0;
    for (int i = threadIdx.x; i < n; i += kThreads) {
        uint32_t att;
        const double x = gg_variate(b, al, k0, k1, tensor_id0 + (uint32_t)s, (uint64_t)(off + i), att);
        worst = max(worst, att);
        if constexpr (sizeof(T) == 4) out[i] = __double2float_rn(x);
        else out[i] = double_to_bf16(x);
    }
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
