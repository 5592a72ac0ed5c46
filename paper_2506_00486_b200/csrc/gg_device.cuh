// Small device helpers shared by the kernels of the library (not installed).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gg {

// 1.5 * 2^23: for |t| < 2^22 the sum t + magic lies in [2^23, 2^24), where the floats are the integers, so
// adding with rounding down gives floor(t) = bits(t +rd magic) - bits(magic).
constexpr uint32_t kMagicBits = 0x4B400000u;

// Shared-memory accesses by 32-bit shared address (one instruction each, no generic-address arithmetic).
__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

// (No memory clobber: the counts are read back only after a barrier, and the clobber would keep the compiler
// from moving the element path's loads across the increment.)
__device__ __forceinline__ void red_inc(uint32_t addr)
{
    asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(addr));
}

__device__ __forceinline__ float rcp_approx(float v)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

// ---- bounds-checking build (-DGG_BOUNDS): every checked global access tests its index against the extent it must
// stay in; a violation is counted (never trapped on) and the access is skipped, so a run of the test suite on such a
// build ends normally and reports how many accesses would have left their buffers.  A normal build compiles the
// checks away.  Each translation unit has its own counter; gg_debug_bounds_violations adds them up.
#ifdef GG_BOUNDS
static __device__ unsigned long long gg_bounds_count;
void gg_register_bounds_reader(unsigned long long (*reader)());
namespace {
unsigned long long gg_bounds_read_this_unit()
{
    unsigned long long v = 0;
    cudaDeviceSynchronize();
    if (cudaMemcpyFromSymbol(&v, gg_bounds_count, sizeof(v)) != cudaSuccess) { cudaGetLastError(); return 0; }
    return v;
}
const int gg_bounds_registered = (gg_register_bounds_reader(&gg_bounds_read_this_unit), 0);
}  // namespace
// true if index i lies in [0, n); else counts the violation
__device__ __forceinline__ bool gg_in_bounds(long long i, long long n)
{
    if (i >= 0 && i < n) return true;
    atomicAdd(&gg_bounds_count, 1ull);
    return false;
}
#define GG_IN_BOUNDS(i, n) gg_in_bounds((long long)(i), (long long)(n))
#else
#define GG_IN_BOUNDS(i, n) true
#endif

// ---- gradient of lambda * R, R the mean k-th order Exponential-Golomb code length of the quantised symbols (Eq. 6-7),
// in the relaxed form of the gradient constrained training section: for an element x of a segment of N elements
//     g = c * sign(x) / (Map(q) + 2^k),   c = lambda * 4 inv / (N ln 2),   q the (clamped) symbol of x,
// and g = 0 where x is zero or nan.  Map is Eq. 6: 0, 1, -1, 2, -2, ... -> 0, 1, 2, 3, 4, ...
// From the symbol: the reciprocal unit plus one Newton step (half an ulp), then the product with c.
__device__ __forceinline__ float eg_grad_of_symbol(int q, float c, uint32_t two_k)
{
    const int n = -q;
    const uint32_t m = ((uint32_t)n << 1) ^ (uint32_t)(n >> 31);      // q > 0: 2q - 1; q < 0: -2q; 0: 0
    const float den = (float)(m + two_k);                              // exact below 2^24
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(den));
    r = fmaf(r, fmaf(-den, r, 1.0f), r);
    return c * r;
}

// The same for any fp32 bit pattern, with the quantiser written out (fp32 product, floor, clamp): the careful path.
__device__ __forceinline__ float eg_grad_exact(uint32_t xb, float inv, int32_t qmin, int32_t qmax, float c, uint32_t two_k)
{
    const float x = __uint_as_float(xb);
    const float t = __fmul_rn(x, inv);
    if (!(t == t) || x == 0.0f) return 0.0f;
    const int q = max(qmin, min(qmax, __float2int_rd(t)));             // floor, saturating, then the clamp
    const float g = eg_grad_of_symbol(q, c, two_k);
    return __uint_as_float(__float_as_uint(g) ^ (xb & 0x80000000u));
}

// Where the vector body of a run starts.  h0: elements up to the first 16-byte boundary of x (the body needs that).
// A warp moves 512 bytes of bf16 input and 1 KB of fp32 gradient per step, and DRAM takes those best as whole blocks:
// a body that starts 16 .. 512 bytes off such a block measured 4 - 20 % slower on long segments.  So the head is
// lengthened, in steps of a 16-byte vector of x, until the gradient (or, without one, x) starts a block of
// `block` bytes: at most block / (bytes a vector covers there) - 1 vectors, handled by the scalar path.
// xe, ge: bytes per element of x and of the gradient; g: the gradient's address at element 0 of the run, or 0.
__device__ __forceinline__ long long aligned_head(long long h0, long long n, unsigned long long x, unsigned long long g, unsigned xe, unsigned ge,
                                                  unsigned block)
{
    const unsigned per_vec = 16u / xe;                                     // elements of a 16-byte vector of x
    const unsigned long long a = g != 0 ? g + (unsigned long long)h0 * ge : x + (unsigned long long)h0 * xe;
    const unsigned step = g != 0 ? per_vec * ge : 16u;                     // bytes the address moves per vector
    const unsigned off = (unsigned)(a & (block - 1u));
    if (off == 0u || (block - off) % step != 0u) return h0 < n ? h0 : n;   // (already there, or never reached in vector steps)
    const long long h = h0 + (long long)((block - off) / step) * per_vec;
    return h <= n ? h : (h0 < n ? h0 : n);
}

// Butterfly sum over the warp: every lane ends with the same bits.
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

}  // namespace gg
