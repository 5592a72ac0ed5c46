// The whole pass for short fp32 segments (gradient rows, fp32 activations): one TEAM of four warps per segment.
// The team loads its segment ONCE into registers (up to 32 elements per thread), takes the moments from there, one
// of its warps inverts the moment ratio and works out the segment's constants, all four build the gradient tables,
// and gradient, penalty and counts are then computed from the registers: DRAM sees the input once and the gradient
// once, and the second pass issues no loads.  Longer segments (up to the short-segment limit) are read a second
// time, from L2.  (Short bf16 segments take the one-warp-per-segment kernel: with 128 elements per lane its
// per-segment work weighs a quarter of what it does here.)
//
//   * gradient: |g| = A[e] * B[j] * (1 + r)^b, e the exponent field, the mantissa cut at seven bits (j) and the rest
//     r < 2^-7 through a degree-4 binomial series; A and B rounded once from fp64, B replicated once per bank (lane
//     l reads word l of row j: no bank conflicts).  A holds NaN for the exponents it does not serve (far from the
//     segment's scale, zero/subnormal, inf/nan, every exponent when |b| > 2); a NaN reaches the vector's penalty
//     partial, whose range check sends the vector to the fp64 evaluation.
//   * histogram: a CTA-wide table, one cell per symbol over [-4096, 4096), serves the segments whose histogram and
//     step equal those of the CTA's first segment; other segments add to global memory element by element.  The
//     CTA's table goes to a scratch slot at the end and a second small kernel adds the slots to the histograms.
#include <cuda_bf16.h>
#include <float.h>

#include "gg_device.cuh"
#include "gg_fit_table.cuh"
#include "gg_internal.h"
#include "gg_small_common.cuh"

namespace gg {
namespace {

constexpr int kTeam = 128;                     // threads of a team
constexpr int kTeamWarps = kTeam / 32;
constexpr int kTeams = 3;                      // teams of a CTA
constexpr int kThreads = kTeam * kTeams;
constexpr int kCtasPerSm = 2;
constexpr int kTabExp = 64;                    // exponents around the segment's scale whose A is evaluated
constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr uint32_t kWinCells = kSymWin;        // symbols [-4096, 4096) of the CTA's table
constexpr uint32_t kSymCells = kWinCells + 2;  // with the two sentinels of the tails
constexpr uint32_t kCntWords = kSymCells;
static_assert(kSymCells + 4 <= (uint32_t)kSmallSlotWords, "scratch slot");

constexpr int kPerVec = 4, kRegVec = 8;        // elements of a 16-byte vector; vectors a thread holds in registers

// What a team shares about its current segment.
struct alignas(16) TeamMem {
    float brep[128 * 32];          // row j: B[j] in every bank (written as 16-byte vectors)
    float a1[256];                 // A[e] as one factor (with lambda's sign), NaN where not served
    float B[128];
    double red[3][kTeamWarps];
    uint32_t bad[kTeamWarps];
    float mn[kTeamWarps], mx[kTeamWarps];
    // constants of the current segment, worked out once by the warp that fits it
    double beta, L, b;             // |g| = 2^(L + b log2|x|)
    unsigned long long *row;       // the segment's histogram, bin 0 = symbol qmin
    float inv;                     // quantiser: q = floor(x * inv)
    float c1, c2, c3, c4;          // fp32 input: binomial coefficients of (1 + r)^b
    uint32_t sign_flip;            // 0x80000000 if lambda < 0 (the tables then hold -|g|)
    int32_t qmin, qmax;
    int active;                    // 0: the gradient is zero everywhere
    int e_lo;                      // first exponent whose A is evaluated
    int series_ok;                 // fp32 input: |b| <= 2
    int hist, fast;                // a histogram is taken; the CTA table serves this segment
};

static_assert(sizeof(TeamMem) % 16 == 0, "every team's tables start on a 16-byte boundary");

struct Smem {
    alignas(16) uint32_t cnt[kCntWords];
    TeamMem team[kTeams];
    double log2m[128];             // log2(1 + j/128): the same for every segment
    // the CTA's histogram key
    int key_hid;
    uint32_t key_inv_bits;
    int key_on;
};

__device__ __forceinline__ void team_sync(int team)
{
    asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "n"(kTeam) : "memory");
}

// Per-segment constants of the branch-free element path (per thread, in registers); everything the cold paths
// need stays in the team's shared memory.
struct SegK {
    float c1, c2, c3, c4;     // fp32 input: binomial coefficients of (1 + r)^b
    float inv;
};

struct Addr {
    uint32_t a, b, cnt;       // shared addresses: A table, this lane's word of B row 0, count cells (fp32: biased, see team_elem)
};

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

// One element given as fp32 bits.  Branch free.  `any` keeps the largest |x * inv| (as float bits) so that one
// compare per vector finds symbols outside the count window; those count on a sentinel.
template <bool GRAD, int HIST>
__device__ __forceinline__ float team_elem(uint32_t xb, const SegK &k, const Addr &ad, const TeamMem &tm, float &mp, uint32_t &any,
                                           uint32_t (&clampc)[2])
{
    float g = 0.0f;
    const uint32_t ax = xb & 0x7FFFFFFFu;
    if constexpr (GRAD) {
        const float a = lds_f32(ad.a + ((ax >> 21) & 0x3FCu));
        const float bj = lds_f32(((ax >> 16) & 127u) * 128u + ad.b);
        const float c = __uint_as_float((ax & 0x007F0000u) | 0x3F800000u);      // 1 + j/128
        const float m = __uint_as_float((ax & 0x007FFFFFu) | 0x3F800000u);
        const float r = (m - c) * rcp_approx(c);                                 // m = c (1 + r), m - c exact
        const float t = r * fmaf(r, fmaf(r, fmaf(r, k.c4, k.c3), k.c2), k.c1);   // (1 + r)^b - 1
        const float ga = a * fmaf(bj, t, bj);
        mp = fmaf(__uint_as_float(ax), fabsf(ga), mp);
        g = __uint_as_float(__float_as_uint(ga) ^ (xb & 0x80000000u));              // the table carries lambda's sign
    }
    if constexpr (HIST == 1) {
        // t clamped to just outside the window: the floor of the clamped value lands on a sentinel for either tail
        // (and for nan, which the maximum replaces by the lower bound)
        const float t = __fmul_rn(__uint_as_float(xb), k.inv);
        any = __float_as_uint(fmaxf(__uint_as_float(any), fabsf(t)));            // (a nan leaves it alone: nan is not counted)
        const float tc = fminf(fmaxf(t, -(float)(kWinCells / 2) - 0.5f), (float)(kWinCells / 2));
        // for |t| < 2^22 the sum lies in [2^23, 2^24) where floats are the integers: rounding down gives floor
        const uint32_t fb = __float_as_uint(__fadd_rd(tc, __uint_as_float(kMagicBits)));
        red_inc((fb << 2) + ad.cnt);
    } else if constexpr (HIST == 2) {
        const int c = count_global(xb, k.inv, tm.qmin, tm.qmax, tm.row);
        if (c) clampc[c - 1] += 1u;
    }
    return g;
}

// (some |x * inv| reached the edge of the window, compared as bit patterns of non-negative floats)
__device__ __forceinline__ bool count_miss(uint32_t any) { return any >= __float_as_uint((float)(kWinCells / 2)); }

// Redo of whatever part of an element the branch-free path could not do; g is its gradient from the first pass.
// grad_bad: the vector's penalty partial is not a finite number, so the whole vector's penalty terms are added
// here instead, in fp64.
template <bool GRAD, int HIST>
__device__ __forceinline__ float team_fix(uint32_t xb, float g, bool grad_bad, const SegK &k, const TeamMem &tm, Smem &sm,
                                          double &pen, uint32_t (&clampc)[2])
{
    const uint32_t ax = xb & 0x7FFFFFFFu;
    if constexpr (GRAD) {
        if (grad_bad) {
            const float a = tm.a1[ax >> 23];
            const double axd = (double)__uint_as_float(ax);
            if (a != a) {     // this element read a NaN marker: the fp64 evaluation
                double gd = 0.0;
                if (tm.active && axd != 0.0) gd = exp2(tm.L + tm.b * log2(axd));
                pen += axd * gd;
                g = __uint_as_float(__float_as_uint((float)gd) ^ tm.sign_flip ^ (xb & 0x80000000u));
            } else {
                pen += axd * (double)fabsf(g);
            }
        }
    }
    if constexpr (HIST == 1) {
        const float t = __fmul_rn(__uint_as_float(xb), k.inv);
        if (t >= (float)(kWinCells / 2) || t < -(float)(kWinCells / 2)) {      // the exact test: floor(t) outside the window
            const int c = count_global(xb, k.inv, tm.qmin, tm.qmax, tm.row);
            if (c) clampc[c - 1] += 1u;
        }
    }
    return g;
}

// fp32 sums of one vector into the fp64 sums of the thread; the vector again in fp64 when a square or a sum left
// the fp32 range or an entry is not finite.
__device__ __forceinline__ void moments_vec(const uint4 &raw, double &s1, double &s2, uint32_t &bad, float &xmin, float &xmax)
{
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    float m1 = 0.0f, m2 = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float x = __uint_as_float(w[i]);
        m1 += fabsf(x);
        m2 = fmaf(x, x, m2);
        xmin = fminf(xmin, x);          // fminf / fmaxf return the non-NaN operand
        xmax = fmaxf(xmax, x);
    }
    if (run_sums_exact_enough(m1, m2)) {
        s1 += (double)m1;
        s2 += (double)m2;
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t am = w[i] & 0x7FFFFFFFu;
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

// Gradient, penalty partial and counts of one vector; the gradient goes to gp (may be null).
template <typename TG, bool GRAD, int HIST>
__device__ __forceinline__ void second_vec(const uint4 &raw, TG *gp, bool accumulate, const SegK &k, const Addr &ad, const TeamMem &tm,
                                           Smem &sm, double &pen, uint32_t (&clampc)[2])
{
    constexpr int N = kPerVec;
    const uint32_t xb[4] = {raw.x, raw.y, raw.z, raw.w};
    float g[N];
    float mp = 0.0f;
    uint32_t any = 0;
#pragma unroll
    for (int i = 0; i < N; ++i) g[i] = team_elem<GRAD, HIST>(xb[i], k, ad, tm, mp, any, clampc);
    // (table products are normal numbers whose terms |x| |g| stay far inside the fp32 range, so a partial that is
    // not finite means a NaN marker was read or an entry is not finite)
    const bool grad_bad = GRAD && !(mp <= FLT_MAX);
    if (grad_bad || (HIST == 1 && count_miss(any))) {
#pragma unroll
        for (int i = 0; i < N; ++i) g[i] = team_fix<GRAD, HIST>(xb[i], g[i], grad_bad, k, tm, sm, pen, clampc);
    }
    if constexpr (GRAD) {
        if (!grad_bad) pen += (double)mp;
        if (gp != nullptr) {
            if constexpr (sizeof(TG) == 4) {
                float4 o = make_float4(g[0], g[1], g[2], g[3]);
                if (accumulate) {
                    const float4 old = *reinterpret_cast<const float4 *>(gp);
                    o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                }
                __stcs(reinterpret_cast<float4 *>(gp), o);
            } else {
                uint32_t o[2];
                const uint32_t *p1 = reinterpret_cast<const uint32_t *>(gp);
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    float lo = g[2 * q], hi = g[2 * q + 1];
                    if (accumulate) {
                        const uint32_t old = p1[q];
                        lo += __uint_as_float(old << 16);
                        hi += __uint_as_float(old & 0xFFFF0000u);
                    }
                    o[q] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
                }
                __stcs(reinterpret_cast<uint2 *>(gp), make_uint2(o[0], o[1]));
            }
        }
    }
}

// Second pass over one segment by its team: the scalar head and tail, then the vectors from the registers (or
// read again, from L2, when the segment did not fit there).
template <typename TG, bool GRAD, int HIST>
__device__ __forceinline__ void second_pass(const float *x, const uint4 *xv, TG *gout, int head, int nvec, int tail0, int n_scalar, bool in_regs,
                                            const uint4 (&reg)[kRegVec], bool accumulate, const SegK &k, const Addr &ad,
                                            const TeamMem &tm, Smem &sm, double &pen, uint32_t (&clampc)[2])
{
    constexpr int EPV = kPerVec, RV = kRegVec;
    if constexpr (!GRAD && HIST == 0) return;     // a fit-only call has no second pass
    const int tt = threadIdx.x % kTeam;
    for (int i = tt; i < n_scalar; i += kTeam) {
        const int idx = i < head ? i : tail0 + (i - head);
        const uint32_t xb = __float_as_uint(__ldg(x + idx));
        float mp = 0.0f;
        uint32_t any = 0;
        float g = team_elem<GRAD, HIST>(xb, k, ad, tm, mp, any, clampc);
        const bool grad_bad = GRAD && !(mp <= FLT_MAX);
        if (grad_bad || (HIST == 1 && count_miss(any))) g = team_fix<GRAD, HIST>(xb, g, grad_bad, k, tm, sm, pen, clampc);
        if constexpr (GRAD) {
            if (!grad_bad) pen += (double)mp;
            if (gout != nullptr) {
                if (accumulate) g += load_grad<TG>(gout + idx);
                store_grad<TG>(gout + idx, g);
            }
        }
    }
    if (in_regs) {
#pragma unroll
        for (int u = 0; u < RV; ++u) {
            const int v = tt + u * kTeam;
            if (v < nvec)
                second_vec<TG, GRAD, HIST>(reg[u], gout != nullptr && GG_IN_BOUNDS(head + v * EPV + EPV - 1, head + nvec * EPV) ? gout + head + v * EPV : nullptr,
                                           accumulate, k, ad, tm, sm, pen, clampc);
        }
    } else {
        // (loads run three vectors ahead of their use)
        uint4 q0 = make_uint4(0u, 0u, 0u, 0u), q1 = q0, q2 = q0;
        if (tt < nvec) q0 = __ldg(xv + tt);
        if (tt + kTeam < nvec) q1 = __ldg(xv + tt + kTeam);
        if (tt + 2 * kTeam < nvec) q2 = __ldg(xv + tt + 2 * kTeam);
        for (int v = tt; v < nvec; v += kTeam) {
            const uint4 raw = q0;
            q0 = q1;
            q1 = q2;
            if (v + 3 * kTeam < nvec) q2 = __ldg(xv + v + 3 * kTeam);
            second_vec<TG, GRAD, HIST>(raw, gout != nullptr ? gout + head + v * EPV : nullptr, accumulate, k, ad, tm, sm, pen, clampc);
        }
    }
}

template <typename TG, bool GRAD, bool HISTK>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) team_kernel(const SmallArgs a)
{
    constexpr int EPV = kPerVec, RV = kRegVec;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31;
    const int team = tid / kTeam, tt = tid % kTeam, tw = tt >> 5;
    const int n_seg = a.map.n_seg;
    const int64_t n_bins = (int64_t)a.qmax - (int64_t)a.qmin + 1;

    if constexpr (HISTK) {
        for (int i = tid; i < (int)kCntWords; i += kThreads) sm.cnt[i] = 0u;
    }
    if (tid < 128) sm.log2m[tid] = log2(1.0 + (double)tid * (1.0 / 128.0));
    if (tid == 0) {
        // the CTA's histogram key: that of the first segment it handles, when steps are given
        sm.key_on = 0;
        sm.key_hid = 0; sm.key_inv_bits = 0u;
        const int s0 = blockIdx.x * kTeams;
        if (HISTK && a.do_hist && !a.step_from_alpha && s0 < n_seg) {
            const float step = a.step[s0];
            sm.key_hid = a.map.hist_id ? a.map.hist_id[s0] : s0;
            sm.key_inv_bits = __float_as_uint((float)(1.0 / (double)step));
            sm.key_on = step > 0.0f && (float)(1.0 / (double)step) < 3.0e38f;
        }
    }
    __syncthreads();
    TeamMem &tm = sm.team[team];
    Addr ad;
    ad.a = (uint32_t)__cvta_generic_to_shared(tm.a1);
    ad.b = (uint32_t)__cvta_generic_to_shared(tm.brep) + (uint32_t)lane * 4u;
    ad.cnt = (uint32_t)__cvta_generic_to_shared(sm.cnt);
    ad.cnt += (kWinCells / 2 + 1 - kMagicBits) << 2;      // cell of symbol q: cnt[q + half + 1], reached from the bits of q + magic

    FitArgs fa{};
    fa.map = a.map;
    fa.beta = a.beta; fa.alpha = a.alpha; fa.sum_abs = a.sum_abs; fa.sum_sq = a.sum_sq; fa.count = a.count; fa.flags = a.flags;
    fa.seed = a.seed; fa.in_dtype_plus1 = (int)GG_F32 + 1;
    fa.step_from_alpha = HISTK && a.do_hist && a.step_from_alpha; fa.step_scale = a.step_scale; fa.step_out = a.step_out;
    fa.hist_on = HISTK && a.do_hist; fa.step = (HISTK && a.do_hist && !a.step_from_alpha) ? a.step : nullptr;
    fa.qmin = a.qmin; fa.qmax = a.qmax;
    const bool accumulate = GRAD && a.accumulate != 0;

    for (int s = blockIdx.x * kTeams + team; s < n_seg; s += gridDim.x * kTeams) {
        const float *x = reinterpret_cast<const float *>(a.map.seg_ptr[s]);
        const int len = (int)a.map.seg_len[s];
        TG *gout = nullptr;
        if constexpr (GRAD) {
            if (a.map.grad_ptr != nullptr) gout = reinterpret_cast<TG *>(a.map.grad_ptr[s]);
        }
        // scalar head up to the first 16-byte boundary of x, 128-bit vector body, scalar tail; if the gradient is
        // not 16-byte aligned at the same element the whole segment is scalar
        int head = (int)(((16u - (uint32_t)(reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / 4u);
        head = min(head, len);
        if (gout != nullptr && (reinterpret_cast<uintptr_t>(gout + head) & 15u) != 0) head = len;
        const int nvec = (len - head) / EPV;
        const int tail0 = head + nvec * EPV;
        const int n_scalar = head + (len - tail0);
        const uint4 *xv = reinterpret_cast<const uint4 *>(x + head);
        const bool in_regs = nvec <= kTeam * RV;

        // ---- the segment into registers (when it fits), and its moments
        uint4 reg[RV];
        if (in_regs) {
#pragma unroll
            for (int u = 0; u < RV; ++u) {
                reg[u] = make_uint4(0u, 0u, 0u, 0u);
                if (tt + u * kTeam < nvec && GG_IN_BOUNDS(head + (tt + u * kTeam) * EPV + EPV - 1, len)) reg[u] = __ldg(xv + tt + u * kTeam);
            }
        }
        double s1 = 0.0, s2 = 0.0;
        uint32_t bad = 0;
        float xmin = INFINITY, xmax = -INFINITY;
        for (int i = tt; i < n_scalar; i += kTeam) {
            const int idx = i < head ? i : tail0 + (i - head);
            const uint32_t xb = __float_as_uint(__ldg(x + idx));
            const uint32_t am = xb & 0x7FFFFFFFu;
            if (am < 0x7F800000u) { s1 += (double)__uint_as_float(am); s2 += (double)__uint_as_float(am) * (double)__uint_as_float(am); }
            else bad += 1u;
            xmin = fminf(xmin, __uint_as_float(xb));
            xmax = fmaxf(xmax, __uint_as_float(xb));
        }
        if (in_regs) {
#pragma unroll
            for (int u = 0; u < RV; ++u)
                if (tt + u * kTeam < nvec) moments_vec(reg[u], s1, s2, bad, xmin, xmax);
        } else {
            for (int v0 = tt; v0 < nvec; v0 += 4 * kTeam) {
                uint4 r4[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (v0 + u * kTeam < nvec) r4[u] = __ldg(xv + v0 + u * kTeam);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (v0 + u * kTeam < nvec) moments_vec(r4[u], s1, s2, bad, xmin, xmax);
            }
        }
        // team reduction in a fixed order: butterfly inside each warp, then the four warps in sequence
        s1 = warp_sum(s1);
        s2 = warp_sum(s2);
        bad = __reduce_add_sync(kFull, bad);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            xmin = fminf(xmin, __shfl_xor_sync(kFull, xmin, o));
            xmax = fmaxf(xmax, __shfl_xor_sync(kFull, xmax, o));
        }
        if (lane == 0) { tm.red[0][tw] = s1; tm.red[1][tw] = s2; tm.bad[tw] = bad; tm.mn[tw] = xmin; tm.mx[tw] = xmax; }
        team_sync(team);

        // ---- fit by the team's first warp (every lane holds the same values), published to the team
        if (tw == 0) {
            s1 = tm.red[0][0]; s2 = tm.red[1][0]; bad = tm.bad[0]; xmin = tm.mn[0]; xmax = tm.mx[0];
#pragma unroll
            for (int w = 1; w < kTeamWarps; ++w) {
                s1 += tm.red[0][w]; s2 += tm.red[1][w]; bad += tm.bad[w];
                xmin = fminf(xmin, tm.mn[w]); xmax = fmaxf(xmax, tm.mx[w]);
            }
            const FitResult fr = fit_finish(fa, s, lane, s1, s2, bad, xmin, xmax);
            // the constants of the second pass, once per segment (every lane computes them, lane 0 publishes)
            const double beta = fr.beta, alpha = fr.alpha;
            const double lam = a.mean_reduction ? a.lambda / (double)max(len, 1) : a.lambda;
            const bool active = GRAD && (beta > 0.0) && (alpha > 0.0) && (lam != 0.0) && (lam == lam);
            const double b = beta - 1.0;
            const double L = active ? log2(fabs(lam) * beta) - beta * log2(alpha) : 0.0;
            // the A table's 64 exponents: 40 binades below the standard deviation's to 23 above
            int e_c = 127;
            if (active) e_c = ilogb(sqrt(s2 / (double)len)) + 127;
            if (lane == 0) {
                tm.beta = beta; tm.L = L; tm.b = b;
                tm.active = active; tm.sign_flip = lam < 0.0 ? 0x80000000u : 0u;
                tm.e_lo = max(1, min(254 - (kTabExp - 1), e_c - 40));
                tm.series_ok = fabs(b) <= 2.0;
                const float bf = (float)b;
                tm.c1 = bf;
                tm.c2 = tm.c1 * (bf - 1.0f) * 0.5f;
                tm.c3 = tm.c2 * (bf - 2.0f) * (1.0f / 3.0f);
                tm.c4 = tm.c3 * (bf - 3.0f) * 0.25f;
                tm.hist = HISTK && a.do_hist != 0;
                if (HISTK && a.do_hist) {
                    const int hid = a.map.hist_id ? a.map.hist_id[s] : s;
                    tm.inv = (float)(1.0 / (double)fr.step);
                    tm.qmin = a.qmin;
                    tm.qmax = a.qmax;
                    tm.row = reinterpret_cast<unsigned long long *>(a.hist) + (int64_t)hid * n_bins;
                    tm.fast = sm.key_on && hid == sm.key_hid && __float_as_uint(tm.inv) == sm.key_inv_bits;
                }
            }
        }
        team_sync(team);

        // ---- the segment's gradient tables, by all threads of the team
        SegK k{};
        if constexpr (GRAD) {
            const bool active = tm.active != 0;
            const double L = tm.L, b = tm.b;
            const int e_lo = tm.e_lo;
            const bool neg = tm.sign_flip != 0u;
            k.c1 = tm.c1; k.c2 = tm.c2; k.c3 = tm.c3; k.c4 = tm.c4;
            for (int e = tt; e < 256; e += kTeam) {
                float v = active ? __int_as_float(0x7FC00000) : 0.0f;
                if (active && tm.series_ok && (uint32_t)(e - e_lo) < (uint32_t)kTabExp) {
                    // one fp32 factor serves if |L + b (e-127)| <= 100: its product with B stays a normal number;
                    // the same bound on L + beta (e-127) keeps the penalty terms |x| |g| normal too
                    const double de = (double)(e - 127);
                    const double e0 = L + b * de;
                    if (fabs(e0) <= 100.0 && fabs(e0 + de) <= 100.0) v = (float)(neg ? -exp2_short(e0) : exp2_short(e0));
                }
                tm.a1[e] = v;
            }
            tm.B[tt] = active ? (float)exp2_short(b * sm.log2m[tt]) : 1.0f;
            team_sync(team);
            // B[j] into every bank of row j: consecutive 16-byte stores, free of bank conflicts
            float4 *rep4 = reinterpret_cast<float4 *>(tm.brep);
#pragma unroll
            for (int q = 0; q < 128 * 32 / 4 / kTeam; ++q) {
                const int i = tt + q * kTeam;
                const float v = tm.B[i >> 3];
                rep4[i] = make_float4(v, v, v, v);
            }
        }
        const bool do_hist = HISTK && tm.hist != 0, fast = do_hist && tm.fast != 0;
        if (do_hist) k.inv = tm.inv;
        team_sync(team);

        // ---- second pass: gradient, penalty partial, counts
        double pen = 0.0;
        uint32_t clampc[2] = {0u, 0u};
        if constexpr (HISTK) {
            if (!do_hist) second_pass<TG, GRAD, 0>(x, xv, gout, head, nvec, tail0, n_scalar, in_regs, reg, accumulate, k, ad, tm, sm, pen, clampc);
            else if (fast) second_pass<TG, GRAD, 1>(x, xv, gout, head, nvec, tail0, n_scalar, in_regs, reg, accumulate, k, ad, tm, sm, pen, clampc);
            else second_pass<TG, GRAD, 2>(x, xv, gout, head, nvec, tail0, n_scalar, in_regs, reg, accumulate, k, ad, tm, sm, pen, clampc);
        } else {
            second_pass<TG, GRAD, 0>(x, xv, gout, head, nvec, tail0, n_scalar, in_regs, reg, accumulate, k, ad, tm, sm, pen, clampc);
        }

        // ---- per-segment results of the second pass
        if constexpr (GRAD) {
            pen = warp_sum(pen);
            if (lane == 0) tm.red[2][tw] = pen;
        }
        if constexpr (HISTK) {
            if (do_hist && a.clamped != nullptr) {
                const uint32_t c0 = __reduce_add_sync(kFull, clampc[0]), c1 = __reduce_add_sync(kFull, clampc[1]);
                const int hid = a.map.hist_id ? a.map.hist_id[s] : s;
                if (lane == 0 && c0) atomicAdd(reinterpret_cast<unsigned long long *>(a.clamped) + 2 * hid, (unsigned long long)c0);
                if (lane == 0 && c1) atomicAdd(reinterpret_cast<unsigned long long *>(a.clamped) + 2 * hid + 1, (unsigned long long)c1);
            }
        }
        team_sync(team);      // (also: everybody is done with the tables before the next segment rewrites them)
        if constexpr (GRAD) {
            if (tt == 0 && a.penalty) {
                double p = 0.0;
                for (int w = 0; w < kTeamWarps; ++w) p += tm.red[2][w];
                // sum |x| |g| = |lambda| beta sum (|x|/alpha)^beta; the penalty carries lambda's sign
                const double beta = tm.beta;
                a.penalty[s] = beta > 0.0 ? (tm.sign_flip ? -p : p) / beta : 0.0;
            }
            team_sync(team);  // (red[2] is written again by the next segment's fit)
        }
    }

    // ---- the CTA's counts go to its slot of the scratch; a flush kernel adds the slots to the histograms
    if constexpr (HISTK) {
        __syncthreads();
        uint32_t *slot = a.cta_counts + (size_t)blockIdx.x * kSmallSlotWords;
        for (uint32_t c = tid; c < kSymCells; c += kThreads) slot[c] = sm.key_on ? sm.cnt[c] : 0u;
        if (tid == 0) {
            slot[kSymCells + 0] = (uint32_t)sm.key_on;
            slot[kSymCells + 1] = (uint32_t)sm.key_hid;
            slot[kSymCells + 2] = sm.key_inv_bits;
            slot[kSymCells + 3] = 0u;
        }
    }
}

template <typename TG>
cudaError_t launch_typed(const SmallArgs &a, int sm_count, cudaStream_t st)
{
    const int grid = team_grid(a.map.n_seg, sm_count);
    auto go = [&](auto kern) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem));
        if (e != cudaSuccess) return e;
        kern<<<grid, kThreads, sizeof(Smem), st>>>(a);
        return cudaGetLastError();
    };
    if (!a.do_hist) return a.do_grad ? go(team_kernel<TG, true, false>) : go(team_kernel<TG, false, false>);
    cudaError_t e = a.do_grad ? go(team_kernel<TG, true, true>) : go(team_kernel<TG, false, true>);
    if (e != cudaSuccess) return e;
    flush_slots_kernel<true><<<(kSymCells + 31) / 32, dim3(32, 8), 0, st>>>(a.cta_counts, grid, a.qmin, a.qmax, a.hist, a.clamped);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_team_f32(gg_dtype grad_dtype, const SmallArgs &a, int sm_count, cudaStream_t st)
{
    if (a.map.n_seg <= 0) return cudaSuccess;
    if (a.do_grad && a.map.grad_ptr != nullptr && grad_dtype == GG_BF16) return launch_typed<uint16_t>(a, sm_count, st);
    return launch_typed<float>(a, sm_count, st);
}

int team_grid(int32_t n_seg, int sm_count)
{
    return (int)min(min((int64_t)(n_seg + kTeams - 1) / kTeams, (int64_t)sm_count * kCtasPerSm), (int64_t)kMaxSlots);
}

}  // namespace gg
