// Per-segment and per-histogram kernels of the GG pass: the fixed-order reduction of the tile
// partials, the moment-ratio inversion (one warp per segment), the penalty sums, and the
// empirical entropy of a count table.  All arithmetic here is fp64; none of it is bandwidth bound.
#include "gg_fit_table.cuh"
#include "gg_device.cuh"
#include "gg_internal.h"

namespace gg {
namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kSegThreads = 256;   // one CTA of 8 warps per segment

// One CTA of eight warps per segment.  The threads sum the tile partials in a fixed order (strided over
// the 256 threads, a butterfly in each warp, the eight warps in sequence, so every thread of warp 0 ends
// with the same bits), then warp 0 inverts the moment ratio: from the context's fit
// table when there is one, else by 33-section search on
// ln(beta): each round the 32 lanes evaluate log_rho at the interior points of the bracket and a
// ballot picks the sub-interval with the sign change; ten rounds shrink [ln .05, ln 20] below
// 1e-14.  The scale follows Eq. 2 with sigma^2 = sum_sq / count.
__global__ void __launch_bounds__(kSegThreads) fit_kernel(const FitArgs a)
{
    __shared__ double sh1[kSegThreads / 32], sh2[kSegThreads / 32];
    __shared__ uint32_t shb[kSegThreads / 32];
    __shared__ float shmn[kSegThreads / 32], shmx[kSegThreads / 32];
    const int s = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t0 = a.map.tile_prefix[s], t1 = a.map.tile_prefix[s + 1];
    double s1 = 0.0, s2 = 0.0;
    uint32_t bad = 0;
    float xmin = INFINITY, xmax = -INFINITY;
#pragma unroll 4
    for (int t = t0 + (int)threadIdx.x; t < t1; t += kSegThreads) {
        s1 += a.part.s1[t];
        s2 += a.part.s2[t];
        bad += a.part.bad[t];
        xmin = fminf(xmin, a.part.xmin[t]);
        xmax = fmaxf(xmax, a.part.xmax[t]);
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    bad = __reduce_add_sync(kFull, bad);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        xmin = fminf(xmin, __shfl_xor_sync(kFull, xmin, o));
        xmax = fmaxf(xmax, __shfl_xor_sync(kFull, xmax, o));
    }
    if (lane == 0) { sh1[warp] = s1; sh2[warp] = s2; shb[warp] = bad; shmn[warp] = xmin; shmx[warp] = xmax; }
    __syncthreads();
    if (warp != 0) return;
    s1 = sh1[0]; s2 = sh2[0]; bad = shb[0]; xmin = shmn[0]; xmax = shmx[0];
    for (int w = 1; w < kSegThreads / 32; ++w) {
        s1 += sh1[w]; s2 += sh2[w]; bad += shb[w];
        xmin = fminf(xmin, shmn[w]); xmax = fmaxf(xmax, shmx[w]);
    }
    fit_finish(a, s, lane, s1, s2, bad, xmin, xmax);
}

// The same with one WARP per segment (eight segments per CTA), for layouts of many segments of few tiles each, where
// a CTA per segment leaves seven of its eight warps idle and the launch takes several waves: lane l adds the tiles
// l, l + 32, ... in order, a butterfly adds the lanes.  (Another order of additions than the kernel above: which of
// the two serves a layout depends on the layout alone, so a layout always gets the same bits.)
__global__ void __launch_bounds__(kSegThreads) fit_warp_kernel(const FitArgs a)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int s = blockIdx.x * (kSegThreads / 32) + warp;
    if (s >= a.map.n_seg) return;
    const int t0 = a.map.tile_prefix[s], t1 = a.map.tile_prefix[s + 1];
    double s1 = 0.0, s2 = 0.0;
    uint32_t bad = 0;
    float xmin = INFINITY, xmax = -INFINITY;
    for (int t = t0 + lane; t < t1; t += 32) {
        s1 += a.part.s1[t];
        s2 += a.part.s2[t];
        bad += a.part.bad[t];
        xmin = fminf(xmin, a.part.xmin[t]);
        xmax = fmaxf(xmax, a.part.xmax[t]);
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    bad = __reduce_add_sync(kFull, bad);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        xmin = fminf(xmin, __shfl_xor_sync(kFull, xmin, o));
        xmax = fmaxf(xmax, __shfl_xor_sync(kFull, xmax, o));
    }
    fit_finish(a, s, lane, s1, s2, bad, xmin, xmax);
}

// penalty[s] = (1/beta_s) * sum over the segment's tiles of sum |x| |g|
//            = lambda_s * sum (|x|/alpha_s)^beta_s   since |x| |g| = lambda beta (|x|/alpha)^beta.
__device__ __forceinline__ void penalty_finalize(const TileMap &map, const TileScratch &part, const double *beta, double *penalty, int s)
{
    __shared__ double shp[kSegThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double p = 0.0;
#pragma unroll 4
    for (int t = map.tile_prefix[s] + (int)threadIdx.x; t < map.tile_prefix[s + 1]; t += kSegThreads) p += part.pen[t];
    p = warp_sum(p);
    if (lane == 0) shp[warp] = p;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kSegThreads / 32; ++w) p += shp[w];      // fixed order
        const double b = beta[s];
        penalty[s] = b > 0.0 ? p / b : 0.0;
    }
}

// Entropy of a count table, H = log2 N - (1/N) sum_{c>0} c log2 c, in two steps so that one large
// table keeps many SMs busy: kEntSplit CTAs per histogram each reduce a slice of the bins to
// (sum c log2 c, sum c) in a fixed order, then one thread per histogram adds the slices in order.
// The slices of a histogram need no second launch: the CTA that finishes a histogram's last slice (a ticket from an
// atomic counter; nobody waits) adds all slices in their fixed order and writes the entropy, then puts the counter
// back to zero for the next call.
constexpr int kEntThreads = 256;
static_assert(kEntThreads == kSegThreads, "one launch serves both");
__device__ __forceinline__ void entropy_slice(const uint64_t *hist, int32_t n_bins, double *part, uint32_t *done, double *entropy_bits, int block)
{
    __shared__ double shAcc[kEntThreads / 32];
    __shared__ unsigned long long shTot[kEntThreads / 32];
    const int h = block / kEntSplit, slice = block % kEntSplit;
    const uint64_t *row = hist + (int64_t)h * n_bins;
    const int per = (n_bins + kEntSplit - 1) / kEntSplit;
    const int k0 = slice * per, k1 = min(n_bins, k0 + per);
    double acc = 0.0;
    unsigned long long tot = 0;
    auto add = [&](uint64_t c) {
        if (c != 0) {
            const double cd = (double)c;
            acc += cd * log2(cd);
            tot += c;
        }
    };
    // (most bins are empty, so the loop is bound by load latency: four independent 16-byte loads, two bins each,
    // per trip when the slice allows; the order in which a thread adds its bins stays fixed)
    if ((reinterpret_cast<uintptr_t>(row + k0) & 15u) == 0 && ((k1 - k0) & 1) == 0) {
        const ulonglong2 *row2 = reinterpret_cast<const ulonglong2 *>(row + k0);
        const int n2 = (k1 - k0) / 2;
        for (int k = threadIdx.x; k < n2; k += 4 * kEntThreads) {
            ulonglong2 c[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) c[u] = k + u * kEntThreads < n2 ? __ldg(row2 + k + u * kEntThreads) : make_ulonglong2(0ull, 0ull);
#pragma unroll
            for (int u = 0; u < 4; ++u) { add(c[u].x); add(c[u].y); }
        }
    } else {
        for (int k = k0 + threadIdx.x; k < k1; k += 4 * kEntThreads) {
            uint64_t c[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) c[u] = k + u * kEntThreads < k1 ? __ldg(row + k + u * kEntThreads) : 0ull;
#pragma unroll
            for (int u = 0; u < 4; ++u) add(c[u]);
        }
    }
    acc = warp_sum(acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(kFull, tot, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { shAcc[warp] = acc; shTot[warp] = tot; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double ra = 0.0;
        unsigned long long rt = 0;
        for (int w = 0; w < kEntThreads / 32; ++w) { ra += shAcc[w]; rt += shTot[w]; }
        part[2 * block] = ra;
        part[2 * block + 1] = (double)rt;      // (exact below 2^53 symbols)
        __threadfence();
        if (atomicAdd(done + h, 1u) == (uint32_t)(kEntSplit - 1)) {
            __threadfence();
            double sa = 0.0, st = 0.0;
            for (int k = 0; k < kEntSplit; ++k) { sa += __ldcg(part + 2 * (h * kEntSplit + k)); st += __ldcg(part + 2 * (h * kEntSplit + k) + 1); }
            entropy_bits[h] = st == 0.0 ? 0.0 : log2(st) - sa / st;
            done[h] = 0u;
        }
    }
}

// What follows the sweeps of a call, in one launch: the first n_ent CTAs take the entropy slices, the others one
// segment's penalty sum each.
__global__ void __launch_bounds__(kSegThreads)
finish_kernel(const TileMap map, const TileScratch part, const double *beta, double *penalty, const uint64_t *hist, int32_t n_bins,
              double *ent_part, uint32_t *ent_done, double *entropy_bits, int n_ent)
{
    if ((int)blockIdx.x < n_ent) entropy_slice(hist, n_bins, ent_part, ent_done, entropy_bits, (int)blockIdx.x);
    else penalty_finalize(map, part, beta, penalty, (int)blockIdx.x - n_ent);
}

}  // namespace

cudaError_t launch_fit(const FitArgs &a, cudaStream_t st)
{
    if (a.map.n_seg <= 0) return cudaSuccess;
    if (a.map.n_seg >= 64 && (int64_t)a.map.n_tiles <= 32 * (int64_t)a.map.n_seg)
        fit_warp_kernel<<<(a.map.n_seg + kSegThreads / 32 - 1) / (kSegThreads / 32), kSegThreads, 0, st>>>(a);
    else
        fit_kernel<<<a.map.n_seg, kSegThreads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_finish(const TileMap &map, const TileScratch &part, const double *beta, double *penalty, int32_t n_pen,
                          const uint64_t *hist, int32_t n_hist, int32_t n_bins, double *entropy_bits, double *scratch,
                          uint32_t *done, cudaStream_t st)
{
    const int n_ent = n_hist > 0 ? n_hist * kEntSplit : 0;
    if (n_ent + n_pen <= 0) return cudaSuccess;
    finish_kernel<<<n_ent + n_pen, kSegThreads, 0, st>>>(map, part, beta, penalty, hist, n_bins, scratch, done, entropy_bits, n_ent);
    return cudaGetLastError();
}

cudaError_t launch_penalty_finalize(const TileMap &map, const TileScratch &part, const double *beta,
                                    double *penalty, cudaStream_t st)
{
    return launch_finish(map, part, beta, penalty, map.n_seg, nullptr, 0, 0, nullptr, nullptr, nullptr, st);
}

cudaError_t launch_entropy(const uint64_t *hist, int32_t n_hist, int32_t n_bins, double *entropy_bits,
                           double *scratch, uint32_t *done, cudaStream_t st)
{
    return launch_finish(TileMap{}, TileScratch{}, nullptr, nullptr, 0, hist, n_hist, n_bins, entropy_bits, scratch, done, st);
}

}  // namespace gg
