// Host side of the library: contexts, cached plans (tile maps + scratch), argument checks and
// the C entry points declared in gg.h.  No kernel lives here.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <memory>
#include <new>
#include <string>
#include <vector>

#include "gg_internal.h"

using namespace gg;

namespace {

constexpr int kMaxPlans = 16;
constexpr int64_t kDefaultChunkBytes = 512ll << 20;

// A plan is everything that depends only on the layout of a call: segment addresses and lengths,
// gradient addresses, histogram ids.  It owns the device tables and the per-tile scratch.
struct Plan {
    std::string key;
    int32_t n_seg = 0, n_tiles = 0;
    void *dev = nullptr;          // one allocation holding all tables and scratch
    TileMap map{};
    TileScratch part{};
    double *params = nullptr;     // [2 * n_seg] device staging for host-supplied (beta, alpha)
    uint64_t last_use = 0;
};

}  // namespace

struct gg_ctx {
    int device = 0;
    std::vector<std::unique_ptr<Plan>> plans;
    uint64_t clock = 0;
    int64_t launches = 0;
    std::string cuda_error;
    // gg_fused_host staging (created on first use)
    struct HostSlot {
        gg_ctx *ctx = nullptr;
        cudaStream_t stream = nullptr;
        void *in = nullptr, *grad = nullptr;
        int64_t in_bytes = 0, grad_bytes = 0;
    } slot[2];
    void *host_dev = nullptr;     // device block for per-segment outputs and histograms
    int64_t host_dev_bytes = 0;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        active = dev;
    }
    ~DeviceGuard() { if (prev >= 0 && prev != active) cudaSetDevice(prev); }
    int active = -1;
};

gg_status cuda_fail(gg_ctx *ctx, cudaError_t e)
{
    if (ctx) ctx->cuda_error = cudaGetErrorString(e);
    cudaGetLastError();   // clear the sticky-free error slot
    return GG_ERR_CUDA;
}

#define GG_CUDA(ctx, call)                                   \
    do {                                                     \
        cudaError_t e__ = (call);                            \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__);\
    } while (0)

inline size_t esize(int dtype) { return dtype == GG_F32 ? 4 : 2; }
inline bool dtype_ok(int dtype) { return dtype == GG_F32 || dtype == GG_BF16; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

gg_status check_segs(const gg_seg *segs, int32_t n_seg, int dtype)
{
    if (n_seg < 0 || (n_seg > 0 && segs == nullptr)) return GG_ERR_INVALID_ARG;
    if (!dtype_ok(dtype)) return GG_ERR_DTYPE;
    int64_t tiles = 0;
    for (int32_t s = 0; s < n_seg; ++s) {
        if (segs[s].len < 0) return GG_ERR_INVALID_ARG;
        if (segs[s].len > 0 && segs[s].ptr == nullptr) return GG_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(segs[s].ptr) % esize(dtype) != 0) return GG_ERR_ALIGNMENT;
        tiles += (segs[s].len + kTile - 1) / kTile;
    }
    if (tiles > 0x7FFFFFFFll) return GG_ERR_WORKSPACE;
    return GG_OK;
}

// Finds or builds the plan for this layout.  Building allocates and uploads with blocking calls.
gg_status get_plan(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, int in_dtype, const gg_seg *grad,
                   int grad_dtype, const int32_t *hist_id, Plan **out)
{
    std::string key;
    key.reserve((size_t)n_seg * 36 + 16);
    const int32_t head[4] = {n_seg, in_dtype, grad ? grad_dtype : -1, hist_id ? 1 : 0};
    key.append(reinterpret_cast<const char *>(head), sizeof(head));
    key.append(reinterpret_cast<const char *>(segs), sizeof(gg_seg) * (size_t)n_seg);
    if (grad) {
        for (int32_t s = 0; s < n_seg; ++s)
            key.append(reinterpret_cast<const char *>(&grad[s].ptr), sizeof(void *));
    }
    if (hist_id) key.append(reinterpret_cast<const char *>(hist_id), sizeof(int32_t) * (size_t)n_seg);

    ctx->clock++;
    for (auto &p : ctx->plans) {
        if (p->key == key) {
            p->last_use = ctx->clock;
            *out = p.get();
            return GG_OK;
        }
    }
    if ((int)ctx->plans.size() >= kMaxPlans) {
        // Evict the least recently used plan.  Work that still uses its tables may be in flight.
        GG_CUDA(ctx, cudaDeviceSynchronize());
        size_t victim = 0;
        for (size_t i = 1; i < ctx->plans.size(); ++i)
            if (ctx->plans[i]->last_use < ctx->plans[victim]->last_use) victim = i;
        cudaFree(ctx->plans[victim]->dev);
        ctx->plans.erase(ctx->plans.begin() + (long)victim);
    }

    std::unique_ptr<Plan> p(new (std::nothrow) Plan);
    if (!p) return GG_ERR_NOMEM;
    p->key = std::move(key);
    p->n_seg = n_seg;
    std::vector<int32_t> prefix((size_t)n_seg + 1, 0);
    for (int32_t s = 0; s < n_seg; ++s)
        prefix[(size_t)s + 1] = prefix[(size_t)s] + (int32_t)((segs[s].len + kTile - 1) / kTile);
    const int32_t n_tiles = prefix[(size_t)n_seg];
    p->n_tiles = n_tiles;

    // layout of the single device block
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t o_ptr = take(sizeof(void *) * (size_t)n_seg);
    const size_t o_gptr = take(sizeof(void *) * (size_t)n_seg);
    const size_t o_len = take(sizeof(int64_t) * (size_t)n_seg);
    const size_t o_pref = take(sizeof(int32_t) * ((size_t)n_seg + 1));
    const size_t o_tseg = take(sizeof(int32_t) * (size_t)n_tiles);
    const size_t o_hid = take(sizeof(int32_t) * (size_t)n_seg);
    const size_t table_bytes = off;
    const size_t o_s1 = take(sizeof(double) * (size_t)n_tiles);
    const size_t o_s2 = take(sizeof(double) * (size_t)n_tiles);
    const size_t o_pen = take(sizeof(double) * (size_t)n_tiles);
    const size_t o_bad = take(sizeof(uint32_t) * (size_t)n_tiles);
    const size_t o_par = take(sizeof(double) * 2 * (size_t)n_seg);
    const size_t total = off > 0 ? off : 256;

    std::vector<char> host(table_bytes > 0 ? table_bytes : 1, 0);
    for (int32_t s = 0; s < n_seg; ++s) {
        reinterpret_cast<const void **>(host.data() + o_ptr)[s] = segs[s].ptr;
        reinterpret_cast<void **>(host.data() + o_gptr)[s] = grad ? grad[s].ptr : nullptr;
        reinterpret_cast<int64_t *>(host.data() + o_len)[s] = segs[s].len;
        reinterpret_cast<int32_t *>(host.data() + o_hid)[s] = hist_id ? hist_id[s] : s;
        for (int32_t t = prefix[(size_t)s]; t < prefix[(size_t)s + 1]; ++t)
            reinterpret_cast<int32_t *>(host.data() + o_tseg)[t] = s;
    }
    memcpy(host.data() + o_pref, prefix.data(), sizeof(int32_t) * prefix.size());

    GG_CUDA(ctx, cudaMalloc(&p->dev, total));
    cudaError_t e = cudaMemcpy(p->dev, host.data(), table_bytes, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { cudaFree(p->dev); return cuda_fail(ctx, e); }
    char *d = static_cast<char *>(p->dev);
    p->map.seg_ptr = reinterpret_cast<const void *const *>(d + o_ptr);
    p->map.grad_ptr = grad ? reinterpret_cast<void *const *>(d + o_gptr) : nullptr;
    p->map.seg_len = reinterpret_cast<const int64_t *>(d + o_len);
    p->map.tile_prefix = reinterpret_cast<const int32_t *>(d + o_pref);
    p->map.tile_seg = reinterpret_cast<const int32_t *>(d + o_tseg);
    p->map.hist_id = reinterpret_cast<const int32_t *>(d + o_hid);
    p->map.n_seg = n_seg;
    p->map.n_tiles = n_tiles;
    p->part.s1 = reinterpret_cast<double *>(d + o_s1);
    p->part.s2 = reinterpret_cast<double *>(d + o_s2);
    p->part.pen = reinterpret_cast<double *>(d + o_pen);
    p->part.bad = reinterpret_cast<uint32_t *>(d + o_bad);
    p->params = reinterpret_cast<double *>(d + o_par);
    p->last_use = ctx->clock;
    *out = p.get();
    ctx->plans.push_back(std::move(p));
    return GG_OK;
}

gg_status check_grad(const gg_seg *segs, const gg_seg *grad, int32_t n_seg, int grad_dtype)
{
    if (!grad) return GG_OK;
    if (!dtype_ok(grad_dtype)) return GG_ERR_DTYPE;
    for (int32_t s = 0; s < n_seg; ++s) {
        if (grad[s].len != segs[s].len) return GG_ERR_INVALID_ARG;
        if (grad[s].len > 0 && grad[s].ptr == nullptr) return GG_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(grad[s].ptr) % esize(grad_dtype) != 0) return GG_ERR_ALIGNMENT;
    }
    return GG_OK;
}

gg_status check_hist(int32_t n_seg, const int32_t *hist_id, int32_t n_hist, int32_t qmin, int32_t qmax)
{
    if (n_hist < 0 || qmax < qmin) return GG_ERR_INVALID_ARG;
    if ((int64_t)qmax - (int64_t)qmin + 1 > (1ll << 24)) return GG_ERR_INVALID_ARG;
    if (hist_id == nullptr) return n_hist == n_seg ? GG_OK : GG_ERR_INVALID_ARG;
    for (int32_t s = 0; s < n_seg; ++s)
        if (hist_id[s] < 0 || hist_id[s] >= n_hist) return GG_ERR_INVALID_ARG;
    return GG_OK;
}

}  // namespace

// ------------------------------------------------------------------------------ C entry points
extern "C" {

int gg_version(void) { return 100; }

const char *gg_status_str(gg_status s)
{
    switch (s) {
    case GG_OK: return "ok";
    case GG_ERR_INVALID_ARG: return "invalid argument";
    case GG_ERR_DTYPE: return "unsupported dtype";
    case GG_ERR_ALIGNMENT: return "pointer not aligned to its element size";
    case GG_ERR_WORKSPACE: return "request exceeds a fixed scratch capacity";
    case GG_ERR_ARCH: return "device is not compute capability 10.x";
    case GG_ERR_CUDA: return "CUDA error";
    case GG_ERR_UNIMPLEMENTED: return "not implemented";
    case GG_ERR_NOMEM: return "out of memory";
    default: return "unknown status";
    }
}

const char *gg_last_cuda_error(const gg_ctx *ctx) { return ctx ? ctx->cuda_error.c_str() : ""; }
int64_t gg_launch_count(const gg_ctx *ctx) { return ctx ? ctx->launches : 0; }

double gg_alpha_from_std(double sigma, double beta)
{
    return sigma * exp(0.5 * (lgamma(1.0 / beta) - lgamma(3.0 / beta)));
}

double gg_init_alpha(int64_t d_in, double xi, double beta)
{
    return sqrt(xi / (double)d_in) * exp(0.5 * (lgamma(1.0 / beta) - lgamma(3.0 / beta)));
}

double gg_diff_entropy_bits(double alpha, double beta)
{
    return (1.0 / beta + log(2.0 * alpha / beta) + lgamma(1.0 / beta)) / log(2.0);
}

gg_status gg_create(gg_ctx **out, int device)
{
    if (!out) return GG_ERR_INVALID_ARG;
    *out = nullptr;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) { cudaGetLastError(); return GG_ERR_CUDA; }
    if (prop.major != 10) return GG_ERR_ARCH;
    gg_ctx *ctx = new (std::nothrow) gg_ctx;
    if (!ctx) return GG_ERR_NOMEM;
    ctx->device = device;
    *out = ctx;
    return GG_OK;
}

gg_status gg_destroy(gg_ctx *ctx)
{
    if (!ctx) return GG_OK;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    for (auto &p : ctx->plans) cudaFree(p->dev);
    for (auto &sl : ctx->slot) {
        if (sl.ctx) gg_destroy(sl.ctx);
        if (sl.stream) cudaStreamDestroy(sl.stream);
        if (sl.in) cudaFree(sl.in);
        if (sl.grad) cudaFree(sl.grad);
    }
    if (ctx->host_dev) cudaFree(ctx->host_dev);
    delete ctx;
    return GG_OK;
}

gg_status gg_fit(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, gg_dtype dtype, double *beta,
                 double *alpha, double *sum_abs, double *sum_sq, int64_t *count, uint32_t *flags,
                 void *stream)
{
    if (!ctx || (n_seg > 0 && (!beta || !alpha))) return GG_ERR_INVALID_ARG;
    gg_status st = check_segs(segs, n_seg, dtype);
    if (st != GG_OK) return st;
    if (n_seg == 0) return GG_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    Plan *p = nullptr;
    st = get_plan(ctx, segs, n_seg, dtype, nullptr, 0, nullptr, &p);
    if (st != GG_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    StreamArgs sa{};
    sa.map = p->map;
    sa.part = p->part;
    GG_CUDA(ctx, launch_stream(kMoments, dtype, GG_F32, false, sa, cs));
    ctx->launches += p->n_tiles > 0;
    FitArgs fa{};
    fa.map = p->map; fa.part = p->part;
    fa.beta = beta; fa.alpha = alpha; fa.sum_abs = sum_abs; fa.sum_sq = sum_sq;
    fa.count = count; fa.flags = flags;
    GG_CUDA(ctx, launch_fit(fa, cs));
    ctx->launches += 1;
    return GG_OK;
}

gg_status gg_penalty_grad(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, gg_dtype in_dtype,
                          const double *beta, const double *alpha, double lambda, int reduction,
                          const gg_seg *grad, gg_dtype grad_dtype, int accumulate, double *penalty,
                          void *stream)
{
    if (!ctx || (n_seg > 0 && (!beta || !alpha))) return GG_ERR_INVALID_ARG;
    if (reduction != GG_SUM && reduction != GG_MEAN) return GG_ERR_INVALID_ARG;
    gg_status st = check_segs(segs, n_seg, in_dtype);
    if (st != GG_OK) return st;
    st = check_grad(segs, grad, n_seg, grad_dtype);
    if (st != GG_OK) return st;
    if (n_seg == 0) return GG_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    Plan *p = nullptr;
    st = get_plan(ctx, segs, n_seg, in_dtype, grad, grad_dtype, nullptr, &p);
    if (st != GG_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    StreamArgs sa{};
    sa.map = p->map; sa.part = p->part;
    sa.beta = beta; sa.alpha = alpha; sa.lambda = lambda;
    sa.mean_reduction = reduction == GG_MEAN; sa.accumulate = accumulate;
    GG_CUDA(ctx, launch_stream(kGrad, in_dtype, grad_dtype, grad != nullptr, sa, cs));
    ctx->launches += p->n_tiles > 0;
    if (penalty) {
        GG_CUDA(ctx, launch_penalty_finalize(p->map, p->part, beta, penalty, cs));
        ctx->launches += 1;
    }
    return GG_OK;
}

gg_status gg_rate_hist(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, gg_dtype dtype,
                       const float *step, const int32_t *hist_id, int32_t n_hist, int32_t qmin,
                       int32_t qmax, uint64_t *hist, int accumulate, double *entropy_bits,
                       uint64_t *clamped_lo_hi, void *stream)
{
    if (!ctx || !hist || (n_seg > 0 && !step)) return GG_ERR_INVALID_ARG;
    gg_status st = check_segs(segs, n_seg, dtype);
    if (st != GG_OK) return st;
    st = check_hist(n_seg, hist_id, n_hist, qmin, qmax);
    if (st != GG_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int32_t n_bins = qmax - qmin + 1;
    if (!accumulate) {
        GG_CUDA(ctx, cudaMemsetAsync(hist, 0, sizeof(uint64_t) * (size_t)n_hist * (size_t)n_bins, cs));
        if (clamped_lo_hi) GG_CUDA(ctx, cudaMemsetAsync(clamped_lo_hi, 0, sizeof(uint64_t) * 2 * (size_t)n_hist, cs));
    }
    if (n_seg > 0) {
        Plan *p = nullptr;
        st = get_plan(ctx, segs, n_seg, dtype, nullptr, 0, hist_id, &p);
        if (st != GG_OK) return st;
        StreamArgs sa{};
        sa.map = p->map; sa.part = p->part;
        sa.step = step; sa.qmin = qmin; sa.qmax = qmax; sa.hist = hist; sa.clamped = clamped_lo_hi;
        GG_CUDA(ctx, launch_stream(kHist, dtype, GG_F32, false, sa, cs));
        ctx->launches += p->n_tiles > 0;
    }
    if (entropy_bits && n_hist > 0) {
        GG_CUDA(ctx, launch_entropy(hist, n_hist, n_bins, entropy_bits, cs));
        ctx->launches += 1;
    }
    return GG_OK;
}

gg_status gg_sample(gg_ctx *ctx, const gg_seg *out, int32_t n_seg, gg_dtype dtype, const double *beta,
                    const double *alpha, uint64_t seed, uint32_t tensor_id0, uint32_t *max_attempts,
                    void *stream)
{
    if (!ctx || (n_seg > 0 && (!beta || !alpha))) return GG_ERR_INVALID_ARG;
    gg_status st = check_segs(out, n_seg, dtype);
    if (st != GG_OK) return st;
    for (int32_t s = 0; s < n_seg; ++s)
        if (!(beta[s] > 0.0) || !(alpha[s] >= 0.0) || !isfinite(beta[s]) || !isfinite(alpha[s]))
            return GG_ERR_INVALID_ARG;
    if (n_seg == 0) return GG_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    Plan *p = nullptr;
    st = get_plan(ctx, out, n_seg, dtype, nullptr, 0, nullptr, &p);
    if (st != GG_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // (beta, alpha) come from pageable host memory: the copy is staged before the call returns
    GG_CUDA(ctx, cudaMemcpyAsync(p->params, beta, sizeof(double) * (size_t)n_seg, cudaMemcpyHostToDevice, cs));
    GG_CUDA(ctx, cudaMemcpyAsync(p->params + n_seg, alpha, sizeof(double) * (size_t)n_seg,
                                 cudaMemcpyHostToDevice, cs));
    if (max_attempts) GG_CUDA(ctx, cudaMemsetAsync(max_attempts, 0, sizeof(uint32_t) * (size_t)n_seg, cs));
    GG_CUDA(ctx, launch_sample(p->map, dtype, p->params, p->params + n_seg, seed, tensor_id0, max_attempts, cs));
    ctx->launches += p->n_tiles > 0;
    return GG_OK;
}

gg_status gg_fused(gg_ctx *ctx, const gg_fused_args *a, void *stream)
{
    if (!ctx || !a) return GG_ERR_INVALID_ARG;
    const int32_t n_seg = a->n_seg;
    if (n_seg > 0 && (!a->beta || !a->alpha)) return GG_ERR_INVALID_ARG;
    if (a->param_mode != GG_PARAMS_FITTED && a->param_mode != GG_PARAMS_GIVEN) return GG_ERR_INVALID_ARG;
    if (a->param_mode == GG_PARAMS_GIVEN && n_seg > 0 && (!a->beta_in || !a->alpha_in)) return GG_ERR_INVALID_ARG;
    if (a->reduction != GG_SUM && a->reduction != GG_MEAN) return GG_ERR_INVALID_ARG;
    if (a->step_mode != GG_STEP_GIVEN && a->step_mode != GG_STEP_FROM_ALPHA) return GG_ERR_INVALID_ARG;
    const bool do_hist = a->hist != nullptr;
    if (do_hist) {
        if (a->step_mode == GG_STEP_FROM_ALPHA &&
            (a->param_mode != GG_PARAMS_FITTED || !a->step_out)) return GG_ERR_INVALID_ARG;
        if (a->step_mode == GG_STEP_GIVEN && n_seg > 0 && !a->step) return GG_ERR_INVALID_ARG;
    }
    gg_status st = check_segs(a->segs, n_seg, a->in_dtype);
    if (st != GG_OK) return st;
    st = check_grad(a->segs, a->grad, n_seg, a->grad_dtype);
    if (st != GG_OK) return st;
    if (do_hist) {
        st = check_hist(n_seg, a->hist_id, a->n_hist, a->qmin, a->qmax);
        if (st != GG_OK) return st;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int32_t n_bins = do_hist ? a->qmax - a->qmin + 1 : 0;
    if (do_hist && !a->accumulate_hist) {
        GG_CUDA(ctx, cudaMemsetAsync(a->hist, 0, sizeof(uint64_t) * (size_t)a->n_hist * (size_t)n_bins, cs));
        if (a->clamped_lo_hi)
            GG_CUDA(ctx, cudaMemsetAsync(a->clamped_lo_hi, 0, sizeof(uint64_t) * 2 * (size_t)a->n_hist, cs));
    }
    if (n_seg > 0) {
        Plan *p = nullptr;
        st = get_plan(ctx, a->segs, n_seg, a->in_dtype, a->grad, a->grad_dtype, do_hist ? a->hist_id : nullptr, &p);
        if (st != GG_OK) return st;
        const gg_dtype in_dt = (gg_dtype)a->in_dtype, g_dt = (gg_dtype)a->grad_dtype;
        const bool want_pg = a->grad != nullptr || a->penalty != nullptr;
        const int tail_flags = (want_pg ? kGrad : 0) | (do_hist ? kHist : 0);

        StreamArgs sa{};
        sa.map = p->map; sa.part = p->part;
        sa.lambda = a->lambda; sa.mean_reduction = a->reduction == GG_MEAN; sa.accumulate = a->accumulate_grad;
        sa.qmin = a->qmin; sa.qmax = a->qmax; sa.hist = a->hist; sa.clamped = a->clamped_lo_hi;
        sa.flags = a->flags;
        FitArgs fa{};
        fa.map = p->map; fa.part = p->part;
        fa.beta = a->beta; fa.alpha = a->alpha; fa.sum_abs = a->sum_abs; fa.sum_sq = a->sum_sq;
        fa.count = a->count; fa.flags = a->flags;
        fa.step_from_alpha = do_hist && a->step_mode == GG_STEP_FROM_ALPHA;
        fa.step_scale = a->step_scale; fa.step_out = a->step_out;

        const double *beta_used;
        if (a->param_mode == GG_PARAMS_FITTED) {
            // sweep 1: moments; fit; sweep 2: gradient + histogram with the fresh parameters
            GG_CUDA(ctx, launch_stream(kMoments, in_dt, g_dt, false, sa, cs));
            GG_CUDA(ctx, launch_fit(fa, cs));
            ctx->launches += 1 + (p->n_tiles > 0);
            sa.beta = a->beta; sa.alpha = a->alpha;
            sa.step = fa.step_from_alpha ? a->step_out : a->step;
            if (tail_flags) {
                GG_CUDA(ctx, launch_stream(tail_flags, in_dt, g_dt, a->grad != nullptr, sa, cs));
                ctx->launches += p->n_tiles > 0;
            }
            beta_used = a->beta;
        } else {
            // one sweep: moments, gradient (given parameters) and histogram together; then the fit,
            // which keeps the clamp bit that the sweep OR-ed into the zeroed flags.
            sa.beta = a->beta_in; sa.alpha = a->alpha_in; sa.step = a->step;
            if (a->flags) {
                GG_CUDA(ctx, cudaMemsetAsync(a->flags, 0, sizeof(uint32_t) * (size_t)n_seg, cs));
                fa.keep_clamp_bit = 1;
            }
            GG_CUDA(ctx, launch_stream(kMoments | tail_flags, in_dt, g_dt, a->grad != nullptr, sa, cs));
            GG_CUDA(ctx, launch_fit(fa, cs));
            ctx->launches += 1 + (p->n_tiles > 0);
            beta_used = a->beta_in;
        }
        if (a->penalty) {
            GG_CUDA(ctx, launch_penalty_finalize(p->map, p->part, beta_used, a->penalty, cs));
            ctx->launches += 1;
        }
    }
    if (do_hist && a->entropy_bits && a->n_hist > 0) {
        GG_CUDA(ctx, launch_entropy(a->hist, a->n_hist, n_bins, a->entropy_bits, cs));
        ctx->launches += 1;
    }
    return GG_OK;
}

gg_status gg_fused_host(gg_ctx *ctx, const gg_fused_args *a, int64_t chunk_bytes)
{
    (void)ctx; (void)a; (void)chunk_bytes;
    return GG_ERR_UNIMPLEMENTED;
}

}  // extern "C"
