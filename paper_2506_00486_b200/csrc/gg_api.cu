// Host side of the library: contexts, cached plans (tile maps + scratch), argument checks and
// the C entry points declared in gg.h.  No kernel lives here.
#include <float.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <memory>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "gg_internal.h"

using namespace gg;

// Readers of the per-unit violation counters of a bounds-checking build (empty in a normal build).
static std::vector<unsigned long long (*)()> &bounds_readers()
{
    static std::vector<unsigned long long (*)()> readers;
    return readers;
}
namespace gg {
void gg_register_bounds_reader(unsigned long long (*reader)()) { bounds_readers().push_back(reader); }
}  // namespace gg

namespace {

constexpr int kMaxPlans = 64;
constexpr int kMaxPlansPerLayout = 16;   // plans of one layout (same lengths, types and histogram ids) that differ in their addresses
// The one-launch fitted pass (off unless switched on by gg_test_hook): a group is what L2 keeps from the first
// read of a tensor to the second while the gradient of the tensor before streams out (measured on B200: about
// 30 MB of 126), and at most one segment per warp of the fitting CTA.
constexpr int64_t kGroupBytes = 28ll << 20;
constexpr int kGroupSegs = 16;
constexpr uint32_t kWaitCap = 1u << 18;     // polls of about 0.5 us each
constexpr int64_t kDefaultChunkBytes = 512ll << 20;     // (256 - 512 MiB measured best: the tail of the last chunk is what is not overlapped)

// A plan is everything that depends only on the layout of a call: segment addresses and lengths,
// gradient addresses, histogram ids.  It owns the device tables and the per-tile scratch.
struct Plan {
    // the layout the plan was built for, compared array by array when a call looks for its plan
    int32_t head[4] = {0, 0, 0, 0};          // n_seg, in_dtype, grad_dtype (-1: none), hist_id given
    std::vector<gg_seg> segs, grad;
    std::vector<int32_t> hist_id;
    int32_t max_hist_id = -1;               // largest entry of hist_id
    int32_t n_seg = 0, n_tiles = 0;
    int64_t max_len = 0;          // longest segment
    int64_t total_len = 0;
    bool aligned16 = true;        // every segment (and gradient segment) starts on a 16-byte boundary
    void *dev = nullptr;          // one allocation holding all tables and scratch
    TileMap map{};
    TileScratch part{};
    double *params = nullptr;     // [2 * n_seg] device staging for host-supplied (beta, alpha)
    double *sd = nullptr;         // [n_seg] standard deviations, written by the fit of a fused call for its second sweep
    // the one-launch fitted pass (bf16 input): groups of consecutive segments and their arrive / ready words
    int4 *groups = nullptr;
    int32_t n_groups = 0;
    uint32_t *sync = nullptr;     // [2 * n_groups]
    uint64_t last_use = 0;
    cudaEvent_t used = nullptr;   // recorded after the last work enqueued with this plan: what an eviction waits for
    // a plan whose layout fits a call with other addresses is pointed at them: the two address tables are uploaded
    // again from this pinned staging block, in stream order
    size_t o_ptr = 0, o_gptr = 0;
    void *pin = nullptr;
    cudaEvent_t repointed = nullptr;   // recorded after the upload: the staging block may be filled again
};

}  // namespace

struct gg_ctx {
    int device = 0;
    int sm_count = 148;
    std::vector<std::unique_ptr<Plan>> plans;
    uint64_t clock = 0;
    int64_t launches = 0;
    int64_t plan_builds = 0, plan_repoints = 0;
    std::string cuda_error;
    double *ent_part = nullptr;   // scratch of the entropy step: 2 * kEntSplit doubles per histogram
    uint32_t *ent_done = nullptr; // and one counter per histogram (zero between calls)
    int64_t ent_hists = 0;
    uint32_t *small_counts = nullptr;   // scratch of the short-segment kernel: one slot of count cells per CTA
    void *chan_buf = nullptr;     // scratch of gg_fused_channels (partials per row block and column)
    int64_t chan_bytes = 0;
    double *seed = nullptr;       // device table that seeds the moment-ratio inversion of the short-segment kernel
    int resident_grid[2][8];      // CTAs the one-launch pass may use, by gradient type and sweep flags (-1: not asked yet)
    bool can_cooperate = false, can_cluster = false;
    int cluster_mode = 0;         // one cluster per segment for medium bf16 segments: 0 never, 1 when the layout suits, 2 whenever it can run
    int cluster_max[5];           // resident clusters of size 1, 2, 4, 8, 16 (-1: not asked yet)
    int resident_mode = 0;        // 1: gg_fused takes the one-launch fitted pass whenever it can run
    int32_t expect_delta = 0;     // test hook: arrivals the fitter waits for beyond the streamers that exist
    uint32_t wait_cap = kWaitCap;
    // optional device timing of the two sweeps of gg_fused (event pairs, summed on read)
    bool timing = false;
    std::vector<cudaEvent_t> ev_first, ev_tail;   // begin, end, begin, end, ...
    std::vector<cudaEvent_t> ev_pool;             // events handed back by gg_timing_read, for the next sweeps
    // gg_fused_host staging (created on first use)
    struct HostSlot {
        gg_ctx *ctx = nullptr;
        cudaStream_t stream = nullptr;
        void *in = nullptr, *grad = nullptr;
        int64_t in_bytes = 0, grad_bytes = 0;
    } slot[2];
    cudaEvent_t host_ready = nullptr, host_done = nullptr;   // join points of the two staging streams
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

// The cached plan of this layout, or null.  A hit costs three memory compares (the most recently used
// plan is tried first), and a layout that hits was validated when its plan was built.
Plan *find_plan(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, int in_dtype, const gg_seg *grad, int grad_dtype,
                const int32_t *hist_id)
{
    const int32_t head[4] = {n_seg, in_dtype, grad ? grad_dtype : -1, hist_id ? 1 : 0};
    Plan *best = nullptr;
    for (auto &p : ctx->plans)       // most recently used first
        if (memcmp(p->head, head, sizeof(head)) == 0 && (best == nullptr || p->last_use > best->last_use)) {
            if (memcmp(p->segs.data(), segs, sizeof(gg_seg) * (size_t)n_seg) != 0) continue;
            if (grad && memcmp(p->grad.data(), grad, sizeof(gg_seg) * (size_t)n_seg) != 0) continue;
            if (hist_id && memcmp(p->hist_id.data(), hist_id, sizeof(int32_t) * (size_t)n_seg) != 0) continue;
            best = p.get();
        }
    if (best) best->last_use = ctx->clock;
    return best;
}

void free_plan(Plan *v)
{
    if (v->used) cudaEventDestroy(v->used);
    if (v->repointed) cudaEventDestroy(v->repointed);
    if (v->pin) cudaFreeHost(v->pin);
    cudaFree(v->dev);
}

// Same lengths, types and histogram ids; the addresses may differ.
bool same_layout(const Plan &p, const int32_t (&head)[4], const gg_seg *segs, int32_t n_seg, const int32_t *hist_id)
{
    if (memcmp(p.head, head, sizeof(head)) != 0) return false;
    for (int32_t s = 0; s < n_seg; ++s)
        if (p.segs[(size_t)s].len != segs[s].len) return false;
    return !hist_id || memcmp(p.hist_id.data(), hist_id, sizeof(int32_t) * (size_t)n_seg) == 0;
}

// Points a plan at other addresses: no allocation on the device and no wait for the device; the upload of the two
// address tables is ordered on `cs` behind the work that still reads the old ones.
gg_status repoint(gg_ctx *ctx, Plan *p, const gg_seg *segs, const gg_seg *grad, cudaStream_t cs)
{
    const size_t n = (size_t)p->n_seg;
    if (p->pin == nullptr) {
        GG_CUDA(ctx, cudaHostAlloc(&p->pin, sizeof(void *) * 2 * n, cudaHostAllocDefault));
        cudaError_t e = cudaEventCreateWithFlags(&p->repointed, cudaEventDisableTiming);
        if (e != cudaSuccess) { cudaFreeHost(p->pin); p->pin = nullptr; p->repointed = nullptr; return cuda_fail(ctx, e); }
    } else {
        GG_CUDA(ctx, cudaEventSynchronize(p->repointed));      // the upload before this one has read the block
    }
    void **tab = static_cast<void **>(p->pin);
    p->aligned16 = true;
    for (size_t s = 0; s < n; ++s) {
        tab[s] = segs[s].ptr;
        tab[n + s] = grad ? grad[s].ptr : nullptr;
        if (reinterpret_cast<uintptr_t>(segs[s].ptr) % 16 != 0 || (grad && reinterpret_cast<uintptr_t>(grad[s].ptr) % 16 != 0))
            p->aligned16 = false;
    }
    char *d = static_cast<char *>(p->dev);
    GG_CUDA(ctx, cudaMemcpyAsync(d + p->o_ptr, tab, sizeof(void *) * n, cudaMemcpyHostToDevice, cs));
    if (grad) GG_CUDA(ctx, cudaMemcpyAsync(d + p->o_gptr, tab + n, sizeof(void *) * n, cudaMemcpyHostToDevice, cs));
    GG_CUDA(ctx, cudaEventRecord(p->repointed, cs));
    p->segs.assign(segs, segs + n);
    if (grad) p->grad.assign(grad, grad + n);
    p->last_use = ctx->clock;
    ctx->plan_repoints++;
    return GG_OK;
}

// Finds or builds the plan for this layout.  Building allocates and uploads with blocking calls; a layout that
// already has kMaxPlansPerLayout plans (or any plan, once the cache is full) gets its least recently used plan
// pointed at the new addresses instead, which neither allocates nor blocks.
gg_status get_plan(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, int in_dtype, const gg_seg *grad,
                   int grad_dtype, const int32_t *hist_id, Plan **out, void *stream)
{
    ctx->clock++;
    if (Plan *hit = find_plan(ctx, segs, n_seg, in_dtype, grad, grad_dtype, hist_id)) {
        *out = hit;
        return GG_OK;
    }
    {
        const int32_t head[4] = {n_seg, in_dtype, grad ? grad_dtype : -1, hist_id ? 1 : 0};
        Plan *lru = nullptr;
        int same = 0;
        for (auto &q : ctx->plans)
            if (same_layout(*q, head, segs, n_seg, hist_id)) {
                ++same;
                if (lru == nullptr || q->last_use < lru->last_use) lru = q.get();
            }
        if (lru != nullptr && (same >= kMaxPlansPerLayout || (int)ctx->plans.size() >= kMaxPlans)) {
            gg_status st = repoint(ctx, lru, segs, grad, static_cast<cudaStream_t>(stream));
            if (st != GG_OK) return st;
            *out = lru;
            return GG_OK;
        }
    }
    if ((int)ctx->plans.size() >= kMaxPlans) {
        // Evict the least recently used plan.  Work that still uses its tables may be in flight: wait for the event
        // recorded after its last use (not for the whole device; an event recorded inside a stream capture cannot
        // be waited for, and then the device is).
        size_t victim = 0;
        for (size_t i = 1; i < ctx->plans.size(); ++i)
            if (ctx->plans[i]->last_use < ctx->plans[victim]->last_use) victim = i;
        Plan *v = ctx->plans[victim].get();
        if (v->used == nullptr || cudaEventSynchronize(v->used) != cudaSuccess) {
            cudaGetLastError();
            GG_CUDA(ctx, cudaDeviceSynchronize());
        }
        free_plan(v);
        ctx->plans.erase(ctx->plans.begin() + (long)victim);
    }

    std::unique_ptr<Plan> p(new (std::nothrow) Plan);
    if (!p) return GG_ERR_NOMEM;
    p->head[0] = n_seg; p->head[1] = in_dtype; p->head[2] = grad ? grad_dtype : -1; p->head[3] = hist_id ? 1 : 0;
    p->segs.assign(segs, segs + n_seg);
    if (grad) p->grad.assign(grad, grad + n_seg);
    if (hist_id) {
        p->hist_id.assign(hist_id, hist_id + n_seg);
        for (int32_t s = 0; s < n_seg; ++s) p->max_hist_id = std::max(p->max_hist_id, hist_id[s]);
    }
    p->n_seg = n_seg;
    std::vector<int32_t> prefix((size_t)n_seg + 1, 0);
    for (int32_t s = 0; s < n_seg; ++s)
        prefix[(size_t)s + 1] = prefix[(size_t)s] + (int32_t)((segs[s].len + kTile - 1) / kTile);
    const int32_t n_tiles = prefix[(size_t)n_seg];
    p->n_tiles = n_tiles;
    for (int32_t s = 0; s < n_seg; ++s) {
        p->max_len = segs[s].len > p->max_len ? segs[s].len : p->max_len;
        p->total_len += segs[s].len;
        if (reinterpret_cast<uintptr_t>(segs[s].ptr) % 16 != 0 || (grad && reinterpret_cast<uintptr_t>(grad[s].ptr) % 16 != 0))
            p->aligned16 = false;
    }

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
    const size_t o_min = take(sizeof(float) * (size_t)n_tiles);
    const size_t o_max = take(sizeof(float) * (size_t)n_tiles);
    const size_t o_par = take(sizeof(double) * 2 * (size_t)n_seg);
    const size_t o_sd = take(sizeof(double) * (size_t)n_seg);
    // groups of the one-launch pass: consecutive segments up to kGroupBytes (a longer segment is alone in its group)
    std::vector<int4> groups;
    if (in_dtype == GG_BF16) {
        for (int32_t s = 0; s < n_seg;) {
            int32_t e = s;
            int64_t bytes = 0;
            while (e < n_seg && e - s < kGroupSegs && (e == s || bytes + segs[e].len * 2 <= kGroupBytes)) bytes += segs[e++].len * 2;
            groups.push_back(make_int4(prefix[(size_t)s], prefix[(size_t)e], s, e));
            s = e;
        }
    }
    const size_t o_grp = take(sizeof(int4) * groups.size());
    const size_t o_sync = take(sizeof(uint32_t) * 2 * groups.size());
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
    if (e == cudaSuccess && !groups.empty())
        e = cudaMemcpy(static_cast<char *>(p->dev) + o_grp, groups.data(), sizeof(int4) * groups.size(), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { cudaFree(p->dev); return cuda_fail(ctx, e); }
    char *d = static_cast<char *>(p->dev);
    p->o_ptr = o_ptr; p->o_gptr = o_gptr;
    ctx->plan_builds++;
    p->groups = reinterpret_cast<int4 *>(d + o_grp);
    p->sync = reinterpret_cast<uint32_t *>(d + o_sync);
    p->n_groups = (int32_t)groups.size();

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
    p->part.xmin = reinterpret_cast<float *>(d + o_min);
    p->part.xmax = reinterpret_cast<float *>(d + o_max);
    p->params = reinterpret_cast<double *>(d + o_par);
    p->sd = reinterpret_cast<double *>(d + o_sd);
    p->last_use = ctx->clock;
    if (cudaEventCreateWithFlags(&p->used, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); p->used = nullptr; }
    *out = p.get();
    ctx->plans.push_back(std::move(p));
    return GG_OK;
}

// After the last launch that uses the plan's tables.
void mark_used(Plan *p, cudaStream_t cs)
{
    if (p != nullptr && p->used != nullptr && cudaEventRecord(p->used, cs) != cudaSuccess) cudaGetLastError();
}

// Brackets one sweep of a fused call: an NVTX range (visible to a profiler that is attached, free otherwise) and,
// when timing is on, a pair of events.
struct SweepTimer {
    gg_ctx *ctx; std::vector<cudaEvent_t> *list; cudaStream_t st; bool on;
    SweepTimer(gg_ctx *c, std::vector<cudaEvent_t> *l, cudaStream_t s) : ctx(c), list(l), st(s), on(c->timing)
    {
        nvtxRangePushA(l == &c->ev_first ? "gg: first sweep (moments, or the whole pass)" : "gg: second sweep (gradient + histogram)");
        if (!on) return;
        cudaEvent_t e = take_event(c);
        if (e == nullptr) { on = false; return; }
        cudaEventRecord(e, st);
        list->push_back(e);
    }
    static cudaEvent_t take_event(gg_ctx *c)
    {
        cudaEvent_t e = nullptr;
        if (!c->ev_pool.empty()) { e = c->ev_pool.back(); c->ev_pool.pop_back(); return e; }
        if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return e;
    }
    ~SweepTimer()
    {
        nvtxRangePop();
        if (!on) return;
        cudaEvent_t e = take_event(ctx);
        if (e == nullptr) { ctx->ev_pool.push_back(list->back()); list->pop_back(); return; }
        cudaEventRecord(e, st);
        list->push_back(e);
    }
};

// Picks the kernel for one sweep: bf16 inputs with a gradient or a histogram take the
// pattern-table kernel, everything else the generic one.
cudaError_t launch_sweep(gg_ctx *ctx, int flags, gg_dtype in_dtype, gg_dtype grad_dtype, bool has_grad_out,
                         const StreamArgs &sa, cudaStream_t cs)
{
    // moments alone: persistent CTAs pay a block reduction per run of tiles instead of one per tile, which wins
    // for long bf16 segments (fp32 input and short segments stream as fast tile by tile)
    if (flags == kMoments && in_dtype == GG_BF16 && (int64_t)sa.map.n_tiles >= 16 * (int64_t)sa.map.n_seg)
        return launch_moments_bf16_sweep(sa, ctx->sm_count, cs);
    if (in_dtype == GG_BF16 && (flags & (kGrad | kHist)) != 0)
        return launch_tail_bf16(flags, grad_dtype, has_grad_out, sa, ctx->sm_count, cs);
    if (in_dtype == GG_F32 && (flags & (kGrad | kHist)) != 0)
        return launch_tail_f32(flags, grad_dtype, has_grad_out, sa, ctx->sm_count, cs);
    return launch_stream(flags, in_dtype, grad_dtype, has_grad_out, sa, cs);
}

// Entropy of n_hist count tables; grows the context's scratch (blocking) the first time a call needs more.
gg_status ensure_entropy_scratch(gg_ctx *ctx, int32_t n_hist)
{
    if (n_hist > ctx->ent_hists) {
        if (ctx->ent_part) {
            GG_CUDA(ctx, cudaDeviceSynchronize());
            cudaFree(ctx->ent_part); cudaFree(ctx->ent_done);
            ctx->ent_part = nullptr; ctx->ent_done = nullptr; ctx->ent_hists = 0;
        }
        GG_CUDA(ctx, cudaMalloc(reinterpret_cast<void **>(&ctx->ent_part), sizeof(double) * 2 * kEntSplit * (size_t)n_hist));
        GG_CUDA(ctx, cudaMalloc(reinterpret_cast<void **>(&ctx->ent_done), sizeof(uint32_t) * (size_t)n_hist));
        GG_CUDA(ctx, cudaMemset(ctx->ent_done, 0, sizeof(uint32_t) * (size_t)n_hist));
        ctx->ent_hists = n_hist;
    }
    return GG_OK;
}

gg_status run_entropy(gg_ctx *ctx, const uint64_t *hist, int32_t n_hist, int32_t n_bins, double *entropy_bits,
                      cudaStream_t cs)
{
    gg_status es = ensure_entropy_scratch(ctx, n_hist);
    if (es != GG_OK) return es;
    GG_CUDA(ctx, launch_entropy(hist, n_hist, n_bins, entropy_bits, ctx->ent_part, ctx->ent_done, cs));
    ctx->launches += 1;
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

// CTAs of the one-launch fitted pass for this kernel variant: all of them must be resident at once, so at most
// what the occupancy of the variant allows, and two per SM.  0 when the pass is switched off or cannot run.
int resident_grid(gg_ctx *ctx, int flags, gg_dtype grad_dtype, bool has_grad_out)
{
    if (ctx->resident_mode == 0 || !ctx->can_cooperate) return 0;
    int &slot = ctx->resident_grid[has_grad_out && grad_dtype == GG_BF16 ? 1 : 0][flags & 7];
    if (slot < 0) {
        int max_grid = 0;
        if (resident_bf16_max_grid(flags, grad_dtype, has_grad_out, ctx->sm_count, &max_grid) != cudaSuccess) {
            cudaGetLastError();
            max_grid = 0;
        }
        slot = std::min(max_grid, 2 * ctx->sm_count);
    }
    return slot;
}

// The cluster size (a power of two up to 16) that stages the longest segment of the plan, or 0 when the
// one-cluster-per-segment kernel does not suit the layout; *n_clusters: clusters to launch.
int cluster_choice(gg_ctx *ctx, const Plan *p, int flags, gg_dtype grad_dtype, bool has_grad_out, int *n_clusters)
{
    if (ctx->cluster_mode == 0 || !ctx->can_cluster || !p->aligned16 || p->n_tiles <= 0) return 0;
    const int64_t per_cta = cluster_tiles_per_cta();
    const int64_t max_tiles = (p->max_len + kTile - 1) / kTile;
    if (max_tiles > 16 * per_cta) return 0;
    int size = 1, slot = 0;
    while ((int64_t)size * per_cta < max_tiles) { size *= 2; ++slot; }
    if (ctx->cluster_mode == 1) {
        // worth it when segments are too long for the short-segment kernels, most of them need the cluster they get
        // (the longest decides its size), and there are clusters enough to fill the GPU
        const int64_t mean_tiles = p->n_tiles / std::max(p->n_seg, 1);
        if (p->max_len <= kSmallSegMax || 2 * mean_tiles < max_tiles || (int64_t)p->n_seg * size < ctx->sm_count) return 0;
    }
    int &cached = ctx->cluster_max[slot];
    if (cached < 0) {
        int n = 0;
        if (cluster_bf16_max_clusters(flags, grad_dtype, has_grad_out, size, &n) != cudaSuccess) { cudaGetLastError(); n = 0; }
        cached = n;
    }
    if (cached <= 0) return 0;
    *n_clusters = std::min(cached, (int)p->n_seg);
    return size;
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

int64_t gg_plan_stats(const gg_ctx *ctx, int32_t what)
{
    if (!ctx) return 0;
    return what == 0 ? ctx->plan_builds : what == 1 ? ctx->plan_repoints : -1;
}

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
    ctx->sm_count = prop.multiProcessorCount;
    for (auto &row : ctx->resident_grid) for (int &v : row) v = -1;
    for (int &v : ctx->cluster_max) v = -1;
    ctx->can_cluster = prop.clusterLaunch != 0;
    ctx->can_cooperate = prop.cooperativeLaunch != 0;
    {
        DeviceGuard guard(device);
        cudaError_t se = guard.ok ? cudaMalloc(reinterpret_cast<void **>(&ctx->seed), sizeof(double) * 2 * (kSeedCells + 1))
                                  : cudaErrorInvalidDevice;
        if (se == cudaSuccess) se = launch_fit_seed_table(ctx->seed, nullptr);
        if (se == cudaSuccess) se = cudaStreamSynchronize(nullptr);
        if (se != cudaSuccess) {
            cudaGetLastError();
            if (ctx->seed) cudaFree(ctx->seed);
            delete ctx;
            return se == cudaErrorMemoryAllocation ? GG_ERR_NOMEM : GG_ERR_CUDA;
        }
    }
    *out = ctx;
    return GG_OK;
}

gg_status gg_destroy(gg_ctx *ctx)
{
    if (!ctx) return GG_OK;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    for (auto &p : ctx->plans) free_plan(p.get());
    for (cudaEvent_t e : ctx->ev_first) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->ev_tail) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
    for (auto &sl : ctx->slot) {
        if (sl.ctx) gg_destroy(sl.ctx);
        if (sl.stream) cudaStreamDestroy(sl.stream);
        if (sl.in) cudaFree(sl.in);
        if (sl.grad) cudaFree(sl.grad);
    }
    if (ctx->host_ready) cudaEventDestroy(ctx->host_ready);
    if (ctx->host_done) cudaEventDestroy(ctx->host_done);
    if (ctx->host_dev) cudaFree(ctx->host_dev);
    if (ctx->seed) cudaFree(ctx->seed);
    if (ctx->small_counts) cudaFree(ctx->small_counts);
    if (ctx->chan_buf) cudaFree(ctx->chan_buf);
    if (ctx->ent_part) cudaFree(ctx->ent_part);
    if (ctx->ent_done) cudaFree(ctx->ent_done);
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
    st = get_plan(ctx, segs, n_seg, dtype, nullptr, 0, nullptr, &p, stream);
    if (st != GG_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    StreamArgs sa{};
    sa.map = p->map;
    sa.part = p->part;
    GG_CUDA(ctx, launch_sweep(ctx, kMoments, dtype, GG_F32, false, sa, cs));
    ctx->launches += p->n_tiles > 0;
    FitArgs fa{};
    fa.map = p->map; fa.part = p->part;
    fa.beta = beta; fa.alpha = alpha; fa.sum_abs = sum_abs; fa.sum_sq = sum_sq;
    fa.count = count; fa.flags = flags; fa.seed = ctx->seed; fa.in_dtype_plus1 = (int)dtype + 1;
    GG_CUDA(ctx, launch_fit(fa, cs));
    ctx->launches += 1;
    mark_used(p, cs);
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
    st = get_plan(ctx, segs, n_seg, in_dtype, grad, grad_dtype, nullptr, &p, stream);
    if (st != GG_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    StreamArgs sa{};
    sa.map = p->map; sa.part = p->part;
    sa.beta = beta; sa.alpha = alpha; sa.lambda = lambda;
    sa.mean_reduction = reduction == GG_MEAN; sa.accumulate = accumulate;
    GG_CUDA(ctx, launch_sweep(ctx, kGrad, in_dtype, grad_dtype, grad != nullptr, sa, cs));
    ctx->launches += p->n_tiles > 0;
    if (penalty) {
        GG_CUDA(ctx, launch_penalty_finalize(p->map, p->part, beta, penalty, cs));
        ctx->launches += 1;
    }
    mark_used(p, cs);
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
        st = get_plan(ctx, segs, n_seg, dtype, nullptr, 0, hist_id, &p, stream);
        if (st != GG_OK) return st;
        StreamArgs sa{};
        sa.map = p->map; sa.part = p->part;
        sa.step = step; sa.qmin = qmin; sa.qmax = qmax; sa.hist = hist; sa.clamped = clamped_lo_hi;
        GG_CUDA(ctx, launch_sweep(ctx, kHist, dtype, GG_F32, false, sa, cs));
        ctx->launches += p->n_tiles > 0;
        mark_used(p, cs);
    }
    if (entropy_bits && n_hist > 0) {
        st = run_entropy(ctx, hist, n_hist, n_bins, entropy_bits, cs);
        if (st != GG_OK) return st;
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
    st = get_plan(ctx, out, n_seg, dtype, nullptr, 0, nullptr, &p, stream);
    if (st != GG_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // (beta, alpha) come from pageable host memory: the copy is staged before the call returns
    GG_CUDA(ctx, cudaMemcpyAsync(p->params, beta, sizeof(double) * (size_t)n_seg, cudaMemcpyHostToDevice, cs));
    GG_CUDA(ctx, cudaMemcpyAsync(p->params + n_seg, alpha, sizeof(double) * (size_t)n_seg,
                                 cudaMemcpyHostToDevice, cs));
    if (max_attempts) GG_CUDA(ctx, cudaMemsetAsync(max_attempts, 0, sizeof(uint32_t) * (size_t)n_seg, cs));
    GG_CUDA(ctx, launch_sample(p->map, dtype, p->params, p->params + n_seg, seed, tensor_id0, max_attempts, cs));
    ctx->launches += p->n_tiles > 0;
    mark_used(p, cs);
    return GG_OK;
}

int64_t gg_debug_bounds_violations(void)
{
#ifdef GG_BOUNDS
    unsigned long long total = 0;
    for (auto reader : bounds_readers()) total += reader();
    return (int64_t)total;
#else
    return -1;
#endif
}

gg_status gg_test_hook(gg_ctx *ctx, int32_t what, int64_t value)
{
    if (!ctx) return GG_ERR_INVALID_ARG;
    switch (what) {
    case GG_HOOK_RESIDENT_MODE:
        if (value < 0 || value > 1) return GG_ERR_INVALID_ARG;
        ctx->resident_mode = (int)value;
        return GG_OK;
    case GG_HOOK_EXTRA_ARRIVALS:
        if (value < 0 || value > 1000) return GG_ERR_INVALID_ARG;
        ctx->expect_delta = (int32_t)value;
        return GG_OK;
    case GG_HOOK_CLUSTER_MODE:
        if (value < 0 || value > 2) return GG_ERR_INVALID_ARG;
        ctx->cluster_mode = (int)value;
        return GG_OK;
    case GG_HOOK_WAIT_CAP:
        if (value < 1 || value > (1ll << 24)) return GG_ERR_INVALID_ARG;
        ctx->wait_cap = (uint32_t)value;
        return GG_OK;
    default: return GG_ERR_INVALID_ARG;
    }
}

gg_status gg_timing_enable(gg_ctx *ctx, int enable)
{
    if (!ctx) return GG_ERR_INVALID_ARG;
    ctx->timing = enable != 0;
    return GG_OK;
}

gg_status gg_timing_read(gg_ctx *ctx, double *ms_first, int64_t *n_first, double *ms_tail, int64_t *n_tail)
{
    if (!ctx) return GG_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    std::vector<cudaEvent_t> *lists[2] = {&ctx->ev_first, &ctx->ev_tail};
    double ms[2] = {0.0, 0.0};
    int64_t cnt[2] = {0, 0};
    gg_status result = GG_OK;
    for (int k = 0; k < 2; ++k) {
        auto &l = *lists[k];
        for (size_t i = 0; i + 1 < l.size(); i += 2) {
            float t = 0.0f;
            cudaError_t e = cudaEventSynchronize(l[i + 1]);
            if (e == cudaSuccess) e = cudaEventElapsedTime(&t, l[i], l[i + 1]);
            if (e != cudaSuccess) result = cuda_fail(ctx, e);
            else { ms[k] += (double)t; cnt[k] += 1; }
        }
        for (cudaEvent_t e : l) ctx->ev_pool.push_back(e);      // (kept for the next sweeps: no event is created per call)
        l.clear();
    }
    if (ms_first) *ms_first = ms[0];
    if (n_first) *n_first = cnt[0];
    if (ms_tail) *ms_tail = ms[1];
    if (n_tail) *n_tail = cnt[1];
    return result;
}

gg_status gg_fused(gg_ctx *ctx, const gg_fused_args *a, void *stream)
{
    if (!ctx || !a) return GG_ERR_INVALID_ARG;
    const int32_t n_seg = a->n_seg;
    if (n_seg > 0 && (!a->beta || !a->alpha)) return GG_ERR_INVALID_ARG;
    if (a->param_mode != GG_PARAMS_FITTED && a->param_mode != GG_PARAMS_GIVEN && a->param_mode != GG_RATE_EG) return GG_ERR_INVALID_ARG;
    const bool eg = a->param_mode == GG_RATE_EG;
    if (a->param_mode == GG_PARAMS_GIVEN && n_seg > 0 && (!a->beta_in || !a->alpha_in)) return GG_ERR_INVALID_ARG;
    if (a->reduction != GG_SUM && a->reduction != GG_MEAN) return GG_ERR_INVALID_ARG;
    if (a->step_mode != GG_STEP_GIVEN && a->step_mode != GG_STEP_FROM_ALPHA) return GG_ERR_INVALID_ARG;
    const bool do_hist = a->hist != nullptr;
    if (do_hist) {
        if (a->step_mode == GG_STEP_FROM_ALPHA &&
            (a->param_mode != GG_PARAMS_FITTED || !a->step_out)) return GG_ERR_INVALID_ARG;
        if (a->step_mode == GG_STEP_GIVEN && n_seg > 0 && !a->step) return GG_ERR_INVALID_ARG;
    }
    // the code-length rate is a function of the symbols: it needs the quantiser of the histogram step
    if (eg && (!do_hist || a->step_mode != GG_STEP_GIVEN || a->eg_k < 0 || a->eg_k > 30)) return GG_ERR_INVALID_ARG;
    // A layout that has a plan was validated when the plan was built: a step that repeats a call pays for
    // three memory compares, not for a walk over its segments.
    gg_status st = GG_OK;
    Plan *p = nullptr;
    if (n_seg > 0 && a->segs && dtype_ok(a->in_dtype) && (!a->grad || dtype_ok(a->grad_dtype))) {
        ctx->clock++;
        p = find_plan(ctx, a->segs, n_seg, a->in_dtype, a->grad, a->grad_dtype, do_hist ? a->hist_id : nullptr);
    }
    if (p == nullptr) {
        st = check_segs(a->segs, n_seg, a->in_dtype);
        if (st != GG_OK) return st;
        st = check_grad(a->segs, a->grad, n_seg, a->grad_dtype);
        if (st != GG_OK) return st;
        if (do_hist) {
            st = check_hist(n_seg, a->hist_id, a->n_hist, a->qmin, a->qmax);
            if (st != GG_OK) return st;
        }
    } else if (do_hist) {
        if (a->n_hist < 0 || a->qmax < a->qmin || (int64_t)a->qmax - (int64_t)a->qmin + 1 > (1ll << 24)) return GG_ERR_INVALID_ARG;
        if (a->hist_id ? p->max_hist_id >= a->n_hist : a->n_hist != n_seg) return GG_ERR_INVALID_ARG;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int32_t n_bins = do_hist ? a->qmax - a->qmin + 1 : 0;
    if (n_seg > 0 && p == nullptr) {
        st = get_plan(ctx, a->segs, n_seg, a->in_dtype, a->grad, a->grad_dtype, do_hist ? a->hist_id : nullptr, &p, stream);
        if (st != GG_OK) return st;
    }
    // The histograms start from zero.  When the call begins with the persistent bf16 moments sweep, that sweep
    // clears them on its way (no memset between two launches); otherwise a memset does.
    const size_t hist_bytes = do_hist ? sizeof(uint64_t) * (size_t)a->n_hist * (size_t)n_bins : 0;
    int n_clusters = 0;
    const int csize = (n_seg > 0 && a->param_mode == GG_PARAMS_FITTED && a->in_dtype == GG_BF16 &&
                       (a->grad != nullptr || a->penalty != nullptr || do_hist) && !(p->max_len <= kSmallSegMax && n_seg >= 64))
                          ? cluster_choice(ctx, p, ((a->grad != nullptr || a->penalty != nullptr) ? kGrad : 0) | (do_hist ? kHist : 0),
                                           (gg_dtype)a->grad_dtype, a->grad != nullptr, &n_clusters)
                          : 0;
    const bool sweep_first = n_seg > 0 && a->param_mode == GG_PARAMS_FITTED && a->in_dtype == GG_BF16 && ctx->resident_mode == 0 &&
                             csize == 0 &&
                             (int64_t)p->n_tiles >= 16 * (int64_t)n_seg &&
                             !(p->max_len <= kSmallSegMax && n_seg >= 64);
    const bool clear_in_sweep = do_hist && !a->accumulate_hist && sweep_first && hist_bytes >= (1u << 20) &&
                                reinterpret_cast<uintptr_t>(a->hist) % 16 == 0 && hist_bytes % 16 == 0;
    if (do_hist && !a->accumulate_hist) {
        if (!clear_in_sweep) GG_CUDA(ctx, cudaMemsetAsync(a->hist, 0, hist_bytes, cs));
        if (a->clamped_lo_hi)
            GG_CUDA(ctx, cudaMemsetAsync(a->clamped_lo_hi, 0, sizeof(uint64_t) * 2 * (size_t)a->n_hist, cs));
    }
    bool entropy_done = false;
    if (n_seg > 0) {
        const gg_dtype in_dt = (gg_dtype)a->in_dtype, g_dt = (gg_dtype)a->grad_dtype;
        const bool want_pg = a->grad != nullptr || a->penalty != nullptr;
        const int tail_flags = (want_pg ? kGrad : 0) | (do_hist ? kHist : 0);

        StreamArgs sa{};
        sa.map = p->map; sa.part = p->part;
        sa.lambda = a->lambda; sa.mean_reduction = a->reduction == GG_MEAN; sa.accumulate = a->accumulate_grad;
        sa.qmin = a->qmin; sa.qmax = a->qmax; sa.hist = a->hist; sa.clamped = a->clamped_lo_hi;
        FitArgs fa{};
        fa.map = p->map; fa.part = p->part;
        fa.beta = a->beta; fa.alpha = a->alpha; fa.sum_abs = a->sum_abs; fa.sum_sq = a->sum_sq;
        fa.count = a->count; fa.flags = a->flags; fa.seed = ctx->seed; fa.in_dtype_plus1 = a->in_dtype + 1;
        fa.step_from_alpha = do_hist && a->step_mode == GG_STEP_FROM_ALPHA;
        fa.step_scale = a->step_scale; fa.step_out = a->step_out;
        fa.hist_on = do_hist; fa.step = a->step; fa.qmin = a->qmin; fa.qmax = a->qmax;

        const double *beta_used;
        // Many short bf16 segments with fitted parameters: one kernel, one warp per segment, does the
        // whole pass (below a few dozen segments the two-sweep path fills the GPU better).
        // (bf16: one warp per segment; fp32: one team of four warps per segment)
        const bool small_path = a->param_mode == GG_PARAMS_FITTED && p->max_len <= kSmallSegMax && n_seg >= 64;
        if (small_path) {
            SmallArgs ka{};
            ka.map = p->map;
            ka.beta = a->beta; ka.alpha = a->alpha; ka.sum_abs = a->sum_abs; ka.sum_sq = a->sum_sq;
            ka.count = a->count; ka.flags = a->flags; ka.penalty = a->penalty;
            ka.lambda = a->lambda; ka.mean_reduction = a->reduction == GG_MEAN; ka.accumulate = a->accumulate_grad;
            ka.do_grad = want_pg; ka.do_hist = do_hist;
            ka.step = a->step; ka.step_from_alpha = fa.step_from_alpha; ka.step_scale = a->step_scale;
            ka.step_out = a->step_out;
            ka.qmin = a->qmin; ka.qmax = a->qmax; ka.hist = a->hist; ka.clamped = a->clamped_lo_hi;
            ka.seed = ctx->seed;
            if (do_hist && ctx->small_counts == nullptr)      // (first use: a blocking allocation, like a plan)
                GG_CUDA(ctx, cudaMalloc(reinterpret_cast<void **>(&ctx->small_counts),
                                        sizeof(uint32_t) * kSmallSlotWords * (size_t)ctx->sm_count * 2));
            ka.cta_counts = ctx->small_counts;
            {
                SweepTimer tm(ctx, &ctx->ev_first, cs);
                if (in_dt == GG_BF16) GG_CUDA(ctx, launch_small_bf16(g_dt, ka, ctx->sm_count, cs));
                else GG_CUDA(ctx, launch_team_f32(g_dt, ka, ctx->sm_count, cs));
            }
            ctx->launches += 1 + (do_hist ? 1 : 0);
        } else if (a->param_mode == GG_PARAMS_FITTED && in_dt == GG_BF16 && tail_flags != 0 &&
                   ctx->resident_mode == 1 && p->n_groups > 0 &&
                   resident_grid(ctx, tail_flags, g_dt, a->grad != nullptr) >= 2) {
            // one launch: every group of segments goes moments -> fit -> gradient + histogram while L2 still holds it
            const int grid = resident_grid(ctx, tail_flags, g_dt, a->grad != nullptr);
            GG_CUDA(ctx, cudaMemsetAsync(p->sync, 0, sizeof(uint32_t) * 2 * (size_t)p->n_groups, cs));
            fa.sd_out = p->sd;
            sa.beta = a->beta; sa.alpha = a->alpha; sa.seg_sd = p->sd;
            sa.step = fa.step_from_alpha ? a->step_out : a->step;
            ResidentArgs ra{};
            ra.groups = p->groups; ra.n_groups = p->n_groups;
            ra.arrive = p->sync; ra.ready = p->sync + p->n_groups;
            ra.expect = (uint32_t)(grid - 1 + ctx->expect_delta);
            ra.wait_cap = ctx->wait_cap;
            ra.keep_tiles = (uint32_t)(kGroupBytes / (kTile * 2));
            ra.fit = fa;
            {
                SweepTimer tm(ctx, &ctx->ev_tail, cs);
                GG_CUDA(ctx, launch_resident_bf16(tail_flags, g_dt, a->grad != nullptr, sa, ra, grid, cs));
            }
            ctx->launches += 1;
            beta_used = a->beta;
        } else if (csize > 0) {
            // one thread-block cluster per segment: the segment is staged in the cluster's shared memory and read from DRAM once
            fa.sd_out = p->sd;
            sa.beta = a->beta; sa.alpha = a->alpha; sa.seg_sd = p->sd;
            sa.step = fa.step_from_alpha ? a->step_out : a->step;
            ClusterArgs ca{};
            ca.fit = fa;
            ca.wait_cap = ctx->wait_cap;
            ca.extra_tx = 16u * (uint32_t)ctx->expect_delta;
            {
                SweepTimer tm(ctx, &ctx->ev_tail, cs);
                GG_CUDA(ctx, launch_cluster_bf16(tail_flags, g_dt, a->grad != nullptr, sa, ca, csize, n_clusters, cs));
            }
            ctx->launches += 1;
            beta_used = a->beta;
        } else if (a->param_mode == GG_PARAMS_FITTED) {
            // sweep 1: moments; fit; sweep 2: gradient + histogram with the fresh parameters
            {
                SweepTimer tm(ctx, &ctx->ev_first, cs);
                if (clear_in_sweep) { sa.zero_ptr = reinterpret_cast<uint4 *>(a->hist); sa.zero_vecs = (int64_t)(hist_bytes / 16); }
                GG_CUDA(ctx, launch_sweep(ctx, kMoments, in_dt, g_dt, false, sa, cs));
                sa.zero_ptr = nullptr; sa.zero_vecs = 0;
            }
            fa.sd_out = p->sd;
            GG_CUDA(ctx, launch_fit(fa, cs));
            ctx->launches += 1 + (p->n_tiles > 0);
            sa.beta = a->beta; sa.alpha = a->alpha; sa.seg_sd = p->sd;
            sa.step = fa.step_from_alpha ? a->step_out : a->step;
            if (tail_flags) {
                SweepTimer tm(ctx, &ctx->ev_tail, cs);
                GG_CUDA(ctx, launch_sweep(ctx, tail_flags, in_dt, g_dt, a->grad != nullptr, sa, cs));
                ctx->launches += p->n_tiles > 0;
            }
            beta_used = a->beta;
        } else if (eg) {
            // one sweep: moments, the gradient of lambda * R (Eq. 7) and the histogram together; then the fit.  The
            // rate itself comes from the histogram afterwards.
            sa.step = a->step; sa.eg_k = a->eg_k;
            {
                SweepTimer tm(ctx, &ctx->ev_first, cs);
                GG_CUDA(ctx, launch_sweep(ctx, kMoments | kHist | (a->grad ? kGrad | kEg : 0), in_dt, g_dt, a->grad != nullptr, sa, cs));
            }
            GG_CUDA(ctx, launch_fit(fa, cs));
            ctx->launches += 1 + (p->n_tiles > 0);
            beta_used = nullptr;
        } else {
            // one sweep: moments, gradient (given parameters) and histogram together; then the fit
            sa.beta = a->beta_in; sa.alpha = a->alpha_in; sa.step = a->step;
            {
                SweepTimer tm(ctx, &ctx->ev_first, cs);
                GG_CUDA(ctx, launch_sweep(ctx, kMoments | tail_flags, in_dt, g_dt, a->grad != nullptr, sa, cs));
            }
            GG_CUDA(ctx, launch_fit(fa, cs));
            ctx->launches += 1 + (p->n_tiles > 0);
            beta_used = a->beta_in;
        }
        // the penalty sums of the segments and the entropy of the histograms: one launch for both
        const bool pen_here = a->penalty && !small_path && !eg;
        if (pen_here && do_hist && a->entropy_bits && a->n_hist > 0) {
            gg_status es = ensure_entropy_scratch(ctx, a->n_hist);
            if (es != GG_OK) return es;
            GG_CUDA(ctx, launch_finish(p->map, p->part, beta_used, a->penalty, n_seg, a->hist, a->n_hist, n_bins, a->entropy_bits,
                                       ctx->ent_part, ctx->ent_done, cs));
            ctx->launches += 1;
            entropy_done = true;
        } else if (pen_here) {
            GG_CUDA(ctx, launch_penalty_finalize(p->map, p->part, beta_used, a->penalty, cs));
            ctx->launches += 1;
        }
        mark_used(p, cs);
    }
    if (do_hist && a->entropy_bits && a->n_hist > 0 && !entropy_done) {
        gg_status es = run_entropy(ctx, a->hist, a->n_hist, n_bins, a->entropy_bits, cs);
        if (es != GG_OK) return es;
    }
    if (eg && a->n_hist > 0 && (a->eg_bits || (a->penalty && n_seg > 0))) {
        // mean code length of every histogram; the penalty of a segment is lambda times that of its histogram
        double *bits = a->eg_bits;
        if (bits == nullptr) {
            gg_status es = ensure_entropy_scratch(ctx, a->n_hist);      // (free again once the entropy kernels above are done)
            if (es != GG_OK) return es;
            bits = ctx->ent_part;
        }
        GG_CUDA(ctx, launch_eg_rate(a->hist, a->n_hist, n_bins, a->qmin, a->eg_k, bits, cs));
        ctx->launches += 1;
        if (a->penalty && n_seg > 0) {
            GG_CUDA(ctx, launch_eg_penalty(bits, p->map.hist_id, a->lambda, a->penalty, n_seg, cs));
            ctx->launches += 1;
        }
    }
    return GG_OK;
}

// Grows a device buffer (never shrinks).  Blocking; the caller has made sure nothing uses it.
static gg_status grow(gg_ctx *ctx, void **buf, int64_t *have, int64_t need)
{
    if (need <= *have) return GG_OK;
    if (*buf) { GG_CUDA(ctx, cudaDeviceSynchronize()); cudaFree(*buf); *buf = nullptr; *have = 0; }
    GG_CUDA(ctx, cudaMalloc(buf, (size_t)need));
    *have = need;
    return GG_OK;
}

gg_status gg_fused_channels(gg_ctx *ctx, const gg_channel_args *a, void *stream)
{
    if (!ctx || !a) return GG_ERR_INVALID_ARG;
    if (!dtype_ok(a->in_dtype)) return GG_ERR_DTYPE;
    const bool f32 = a->in_dtype == GG_F32;
    if (a->rows < 0 || a->cols < 0 || a->ld < a->cols) return GG_ERR_INVALID_ARG;
    if (a->cols > 0 && (!a->beta || !a->alpha)) return GG_ERR_INVALID_ARG;
    if (a->rows > 0 && a->cols > 0 && !a->x) return GG_ERR_INVALID_ARG;
    if (a->reduction != GG_SUM && a->reduction != GG_MEAN) return GG_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(a->x) % esize(a->in_dtype) != 0) return GG_ERR_ALIGNMENT;
    if (a->grad) {
        if (!dtype_ok(a->grad_dtype)) return GG_ERR_DTYPE;
        if (a->grad_ld < a->cols) return GG_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(a->grad) % esize(a->grad_dtype) != 0) return GG_ERR_ALIGNMENT;
    }
    const bool do_hist = a->hist != nullptr;
    if (do_hist) {
        if (a->qmax < a->qmin || (int64_t)a->qmax - (int64_t)a->qmin + 1 > (1ll << 24)) return GG_ERR_INVALID_ARG;
        if (!(a->step > 0.0f) || !(a->step <= FLT_MAX)) return GG_ERR_INVALID_ARG;
    }
    const int64_t n_mom = (a->rows + kChanMomRows - 1) / kChanMomRows;
    if (n_mom > 65535 || a->cols > (1ll << 31) - kChanStrip) return GG_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int32_t n_bins = do_hist ? a->qmax - a->qmin + 1 : 0;
    if (do_hist && !a->accumulate_hist) {
        GG_CUDA(ctx, cudaMemsetAsync(a->hist, 0, sizeof(uint64_t) * (size_t)n_bins, cs));
        if (a->clamped_lo_hi) GG_CUDA(ctx, cudaMemsetAsync(a->clamped_lo_hi, 0, sizeof(uint64_t) * 2, cs));
    }
    if (a->cols > 0) {
        const bool want_pg = a->grad != nullptr || a->penalty != nullptr;
        ChanArgs ka{};
        ka.x = static_cast<const uint16_t *>(a->x);
        ka.rows = a->rows; ka.cols = a->cols; ka.ld = a->ld; ka.in_f32 = f32 ? 1 : 0;
        ka.grad = a->grad; ka.grad_ld = a->grad_ld; ka.accumulate = a->accumulate_grad;
        ka.n_mom_blocks = (int32_t)n_mom;
        ka.n_slices = chan_slices(a->rows, a->cols, ctx->sm_count, f32 ? kChanStripF32 : kChanStrip);
        // scratch: doubles first, then the 32-bit arrays
        const size_t nc = (size_t)a->cols, nm = (size_t)n_mom * nc, ns = (size_t)ka.n_slices * nc;
        // table space in units of a narrow (fp32) strip: a wide (bf16) strip takes two
        const size_t n_strips = 2 * ((nc + kChanStrip - 1) / kChanStrip);
        const size_t n_dbl = 2 * nm + 2 * nc + ns, n_w32 = 3 * nm + 2 * nc + n_strips * (kChanTabFloats / 2 + 1) + 8;
        void *buf = ctx->chan_buf;
        gg_status st = grow(ctx, &buf, &ctx->chan_bytes, (int64_t)(n_dbl * 8 + n_w32 * 4));
        ctx->chan_buf = buf;
        if (st != GG_OK) return st;
        double *d = static_cast<double *>(ctx->chan_buf);
        ka.s1 = d; ka.s2 = d + nm; ka.L = d + 2 * nm; ka.b = ka.L + nc; ka.pen = ka.b + nc;
        uint32_t *w = reinterpret_cast<uint32_t *>(d + n_dbl);
        ka.bad = w;
        ka.xmin = reinterpret_cast<float *>(w + nm);
        ka.xmax = reinterpret_cast<float *>(w + 2 * nm);
        ka.amax = reinterpret_cast<float *>(w + 3 * nm);
        ka.sd = reinterpret_cast<float *>(w + 3 * nm + nc);
        ka.tab_elo = reinterpret_cast<int32_t *>(w + 3 * nm + 2 * nc);
        // (the tables are copied as 16-byte vectors: n_dbl * 8 is a multiple of 16 only if n_dbl is even)
        ka.tab = reinterpret_cast<float *>(w + (3 * nm + 2 * nc + n_strips + 3) / 4 * 4 + (n_dbl & 1) * 2);
        ka.beta = a->beta; ka.alpha = a->alpha; ka.sum_abs = a->sum_abs; ka.sum_sq = a->sum_sq;
        ka.count = a->count; ka.flags = a->flags; ka.penalty = a->penalty;
        ka.seed = ctx->seed;
        ka.lambda = a->reduction == GG_MEAN && a->rows > 0 ? a->lambda / (double)a->rows : a->lambda;
        ka.do_grad = want_pg; ka.do_hist = do_hist;
        ka.step = a->step; ka.qmin = a->qmin; ka.qmax = a->qmax; ka.hist = a->hist; ka.clamped = a->clamped_lo_hi;
        {
            SweepTimer tm(ctx, &ctx->ev_first, cs);
            GG_CUDA(ctx, f32 ? launch_chan_moments_f32(ka, cs) : launch_chan_moments(ka, cs));
        }
        GG_CUDA(ctx, launch_chan_fit(ka, cs));
        ctx->launches += 1 + (a->rows > 0);
        if ((want_pg || do_hist) && a->rows > 0) {
            SweepTimer tm(ctx, &ctx->ev_tail, cs);
            GG_CUDA(ctx, f32 ? launch_chan_tail_f32((gg_dtype)a->grad_dtype, ka, ctx->sm_count, cs)
                             : launch_chan_tail((gg_dtype)a->grad_dtype, ka, ctx->sm_count, cs));
            ctx->launches += 1 + (want_pg ? 1 : 0);
        }
        if (a->penalty) {
            if (a->rows <= 0) GG_CUDA(ctx, cudaMemsetAsync(a->penalty, 0, sizeof(double) * nc, cs));
            else { GG_CUDA(ctx, launch_chan_penalty(ka, cs)); ctx->launches += 1; }
        }
    }
    if (do_hist && a->entropy_bits) {
        gg_status es = run_entropy(ctx, a->hist, 1, n_bins, a->entropy_bits, cs);
        if (es != GG_OK) return es;
    }
    return GG_OK;
}

gg_status gg_fused_host(gg_ctx *ctx, const gg_fused_args *a, int64_t chunk_bytes)
{
    if (!ctx || !a) return GG_ERR_INVALID_ARG;
    const int32_t n_seg = a->n_seg;
    if (n_seg > 0 && (!a->beta || !a->alpha)) return GG_ERR_INVALID_ARG;
    if (a->param_mode != GG_PARAMS_FITTED && a->param_mode != GG_PARAMS_GIVEN) return GG_ERR_INVALID_ARG;      // (GG_RATE_EG: device buffers only)
    if (a->param_mode == GG_PARAMS_GIVEN && n_seg > 0 && (!a->beta_in || !a->alpha_in)) return GG_ERR_INVALID_ARG;
    if (a->step_mode != GG_STEP_GIVEN && a->step_mode != GG_STEP_FROM_ALPHA) return GG_ERR_INVALID_ARG;
    const bool do_hist = a->hist != nullptr;
    if (do_hist) {
        if (a->step_mode == GG_STEP_FROM_ALPHA && (a->param_mode != GG_PARAMS_FITTED || !a->step_out))
            return GG_ERR_INVALID_ARG;
        if (a->step_mode == GG_STEP_GIVEN && n_seg > 0 && !a->step) return GG_ERR_INVALID_ARG;
        gg_status hs = check_hist(n_seg, a->hist_id, a->n_hist, a->qmin, a->qmax);
        if (hs != GG_OK) return hs;
    }
    gg_status st = check_segs(a->segs, n_seg, a->in_dtype);
    if (st != GG_OK) return st;
    st = check_grad(a->segs, a->grad, n_seg, a->grad_dtype);
    if (st != GG_OK) return st;
    if (chunk_bytes <= 0) chunk_bytes = kDefaultChunkBytes;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;

    const size_t es = esize(a->in_dtype), gs = a->grad ? esize(a->grad_dtype) : 0;
    // chunks of whole consecutive segments; each segment starts on a 256-byte boundary of the stage
    struct Chunk { int32_t s0, s1; };
    std::vector<Chunk> chunks;
    std::vector<int64_t> in_off((size_t)n_seg), g_off((size_t)n_seg);
    int64_t max_in = 0, max_g = 0;
    for (int32_t s = 0; s < n_seg;) {
        int64_t ib = 0, gb = 0;
        int32_t e = s;
        while (e < n_seg) {
            const int64_t add = (int64_t)align_up((size_t)a->segs[e].len * es, 256);
            if (e > s && ib + add > chunk_bytes) break;
            in_off[(size_t)e] = ib; g_off[(size_t)e] = gb;
            ib += add;
            gb += (int64_t)align_up((size_t)a->segs[e].len * gs, 256);
            ++e;
        }
        chunks.push_back({s, e});
        if (ib > max_in) max_in = ib;
        if (gb > max_g) max_g = gb;
        s = e;
    }

    for (auto &sl : ctx->slot) {
        if (!sl.ctx) { st = gg_create(&sl.ctx, ctx->device); if (st != GG_OK) return st; }
        if (!sl.stream) GG_CUDA(ctx, cudaStreamCreateWithFlags(&sl.stream, cudaStreamNonBlocking));
        st = grow(ctx, &sl.in, &sl.in_bytes, max_in > 0 ? max_in : 256);
        if (st != GG_OK) return st;
        if (a->grad) { st = grow(ctx, &sl.grad, &sl.grad_bytes, max_g > 0 ? max_g : 256); if (st != GG_OK) return st; }
    }
    // device block for per-segment results and histograms
    const int64_t n_bins = do_hist ? (int64_t)a->qmax - a->qmin + 1 : 0;
    const int32_t n_hist = do_hist ? a->n_hist : 0;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t nd = (size_t)n_seg;
    const size_t o_beta = take(8 * nd), o_alpha = take(8 * nd), o_s1 = take(8 * nd), o_s2 = take(8 * nd);
    const size_t o_cnt = take(8 * nd), o_flags = take(4 * nd), o_pen = take(8 * nd), o_step = take(4 * nd);
    const size_t o_bin = take(8 * nd), o_ain = take(8 * nd);
    const size_t o_hist = take(8 * (size_t)n_hist * (size_t)n_bins), o_ent = take(8 * (size_t)n_hist);
    const size_t o_cl = take(16 * (size_t)n_hist);
    st = grow(ctx, &ctx->host_dev, &ctx->host_dev_bytes, (int64_t)(off > 0 ? off : 256));
    if (st != GG_OK) return st;
    char *d = static_cast<char *>(ctx->host_dev);
    cudaStream_t s0 = ctx->slot[0].stream, s1 = ctx->slot[1].stream;

    // inputs that every chunk needs, and the histogram's starting state, on stream 0
    if (a->param_mode == GG_PARAMS_GIVEN && n_seg > 0) {
        GG_CUDA(ctx, cudaMemcpyAsync(d + o_bin, a->beta_in, 8 * nd, cudaMemcpyHostToDevice, s0));
        GG_CUDA(ctx, cudaMemcpyAsync(d + o_ain, a->alpha_in, 8 * nd, cudaMemcpyHostToDevice, s0));
    }
    if (do_hist && a->step_mode == GG_STEP_GIVEN && n_seg > 0)
        GG_CUDA(ctx, cudaMemcpyAsync(d + o_step, a->step, 4 * nd, cudaMemcpyHostToDevice, s0));
    if (do_hist) {
        const size_t hb = 8 * (size_t)n_hist * (size_t)n_bins;
        if (a->accumulate_hist) {
            GG_CUDA(ctx, cudaMemcpyAsync(d + o_hist, a->hist, hb, cudaMemcpyHostToDevice, s0));
            if (a->clamped_lo_hi)
                GG_CUDA(ctx, cudaMemcpyAsync(d + o_cl, a->clamped_lo_hi, 16 * (size_t)n_hist, cudaMemcpyHostToDevice, s0));
            else
                GG_CUDA(ctx, cudaMemsetAsync(d + o_cl, 0, 16 * (size_t)n_hist, s0));
        } else {
            GG_CUDA(ctx, cudaMemsetAsync(d + o_hist, 0, hb, s0));
            GG_CUDA(ctx, cudaMemsetAsync(d + o_cl, 0, 16 * (size_t)n_hist, s0));
        }
    }
    if (ctx->host_ready == nullptr) GG_CUDA(ctx, cudaEventCreateWithFlags(&ctx->host_ready, cudaEventDisableTiming));
    if (ctx->host_done == nullptr) GG_CUDA(ctx, cudaEventCreateWithFlags(&ctx->host_done, cudaEventDisableTiming));
    cudaEvent_t ready = ctx->host_ready, done1 = ctx->host_done;
    gg_status result = GG_OK;
    cudaError_t ce = cudaEventRecord(ready, s0);
    if (ce == cudaSuccess) ce = cudaStreamWaitEvent(s1, ready, 0);
    if (ce != cudaSuccess) result = cuda_fail(ctx, ce);

    std::vector<gg_seg> dsegs, dgrad;
    std::vector<int32_t> hid;
    for (size_t c = 0; c < chunks.size() && result == GG_OK; ++c) {
        auto &sl = ctx->slot[c & 1];
        const int32_t b = chunks[c].s0, e = chunks[c].s1, m = e - b;
        dsegs.resize((size_t)m); dgrad.resize((size_t)m); hid.resize((size_t)m);
        for (int32_t s = b; s < e && result == GG_OK; ++s) {
            char *din = static_cast<char *>(sl.in) + in_off[(size_t)s];
            dsegs[(size_t)(s - b)] = gg_seg{din, a->segs[s].len};
            if (a->segs[s].len > 0) {
                ce = cudaMemcpyAsync(din, a->segs[s].ptr, (size_t)a->segs[s].len * es, cudaMemcpyHostToDevice, sl.stream);
                if (ce != cudaSuccess) result = cuda_fail(ctx, ce);
            }
            if (a->grad) {
                char *dg = static_cast<char *>(sl.grad) + g_off[(size_t)s];
                dgrad[(size_t)(s - b)] = gg_seg{dg, a->segs[s].len};
                if (a->accumulate_grad && a->segs[s].len > 0 && result == GG_OK) {
                    ce = cudaMemcpyAsync(dg, a->grad[s].ptr, (size_t)a->segs[s].len * gs, cudaMemcpyHostToDevice, sl.stream);
                    if (ce != cudaSuccess) result = cuda_fail(ctx, ce);
                }
            }
            hid[(size_t)(s - b)] = a->hist_id ? a->hist_id[s] : s;
        }
        if (result != GG_OK) break;
        gg_fused_args sub = *a;
        sub.segs = dsegs.data(); sub.n_seg = m;
        sub.beta = reinterpret_cast<double *>(d + o_beta) + b;
        sub.alpha = reinterpret_cast<double *>(d + o_alpha) + b;
        sub.sum_abs = reinterpret_cast<double *>(d + o_s1) + b;
        sub.sum_sq = reinterpret_cast<double *>(d + o_s2) + b;
        sub.count = reinterpret_cast<int64_t *>(d + o_cnt) + b;
        sub.flags = reinterpret_cast<uint32_t *>(d + o_flags) + b;
        sub.beta_in = reinterpret_cast<const double *>(d + o_bin) + b;
        sub.alpha_in = reinterpret_cast<const double *>(d + o_ain) + b;
        sub.grad = a->grad ? dgrad.data() : nullptr;
        sub.penalty = a->penalty ? reinterpret_cast<double *>(d + o_pen) + b : nullptr;
        sub.step = reinterpret_cast<const float *>(d + o_step) + b;
        sub.step_out = reinterpret_cast<float *>(d + o_step) + b;
        if (do_hist) {
            sub.hist_id = hid.data();
            sub.hist = reinterpret_cast<uint64_t *>(d + o_hist);
            sub.accumulate_hist = 1;
            sub.entropy_bits = nullptr;
            sub.clamped_lo_hi = reinterpret_cast<uint64_t *>(d + o_cl);
        }
        const int64_t before = sl.ctx->launches;
        result = gg_fused(sl.ctx, &sub, sl.stream);
        ctx->launches += sl.ctx->launches - before;
        if (result == GG_ERR_CUDA) ctx->cuda_error = sl.ctx->cuda_error;
        for (int32_t s = b; s < e && result == GG_OK && a->grad; ++s) {
            if (a->segs[s].len == 0) continue;
            ce = cudaMemcpyAsync(a->grad[s].ptr, static_cast<char *>(sl.grad) + g_off[(size_t)s],
                                 (size_t)a->segs[s].len * gs, cudaMemcpyDeviceToHost, sl.stream);
            if (ce != cudaSuccess) result = cuda_fail(ctx, ce);
        }
    }
    // join stream 1 into stream 0, finish the histogram statistics, bring the results back
    if (result == GG_OK) {
        ce = cudaEventRecord(done1, s1);
        if (ce == cudaSuccess) ce = cudaStreamWaitEvent(s0, done1, 0);
        if (ce == cudaSuccess && do_hist && a->entropy_bits && n_hist > 0) {
            if (run_entropy(ctx, reinterpret_cast<uint64_t *>(d + o_hist), n_hist, (int32_t)n_bins,
                            reinterpret_cast<double *>(d + o_ent), s0) != GG_OK)
                ce = cudaErrorUnknown;
        }
        auto back = [&](void *host, size_t o, size_t bytes) {
            if (ce == cudaSuccess && host && bytes) ce = cudaMemcpyAsync(host, d + o, bytes, cudaMemcpyDeviceToHost, s0);
        };
        back(a->beta, o_beta, 8 * nd); back(a->alpha, o_alpha, 8 * nd);
        back(a->sum_abs, o_s1, 8 * nd); back(a->sum_sq, o_s2, 8 * nd);
        back(a->count, o_cnt, 8 * nd); back(a->flags, o_flags, 4 * nd);
        back(a->penalty, o_pen, 8 * nd);
        if (do_hist) {
            if (a->step_mode == GG_STEP_FROM_ALPHA) back(a->step_out, o_step, 4 * nd);
            back(a->hist, o_hist, 8 * (size_t)n_hist * (size_t)n_bins);
            back(a->entropy_bits, o_ent, 8 * (size_t)n_hist);
            back(a->clamped_lo_hi, o_cl, 16 * (size_t)n_hist);
        }
        if (ce != cudaSuccess) result = cuda_fail(ctx, ce);
    }
    // always drain both streams before returning: host buffers are the caller's again
    cudaError_t e0 = cudaStreamSynchronize(s0), e1 = cudaStreamSynchronize(s1);
    if (result == GG_OK && e0 != cudaSuccess) result = cuda_fail(ctx, e0);
    if (result == GG_OK && e1 != cudaSuccess) result = cuda_fail(ctx, e1);
    return result;
}

}  // extern "C"

// ------------------------------------------------------------------ code lengths and the GCT step

namespace {

// Index of the highest set bit of v (v > 0).
inline int top_bit(uint64_t v) { return 63 - __builtin_clzll(v); }

// Average Huffman code length of the occupied bins of one count table.  The tree is grown with a binary
// min-heap of (weight, node): the two lightest nodes get a common parent until one root is left.  A parent
// is always created after its children, so one pass from the root down the node numbers gives every depth;
// the code length of a symbol is the depth of its leaf and the total sum(count * length) stays an integer
// (128 bits wide: counts go up to 2^63 and depths up to the number of leaves).
struct HuffmanScratch {
    std::vector<uint64_t> weight;
    std::vector<uint32_t> up, depth;
    std::vector<std::pair<uint64_t, uint32_t>> heap;
};

double huffman_bits(const uint64_t *row, int64_t n_bins, HuffmanScratch &w)
{
    w.weight.clear();
    for (int64_t b = 0; b < n_bins; ++b)
        if (row[b] != 0) w.weight.push_back(row[b]);
    const uint32_t n_leaf = (uint32_t)w.weight.size();
    if (n_leaf < 2) return 0.0;
    const uint32_t n_node = 2 * n_leaf - 1;
    w.weight.resize(n_node);
    w.up.assign(n_node, n_node);
    w.heap.clear();
    for (uint32_t i = 0; i < n_leaf; ++i) w.heap.emplace_back(w.weight[i], i);
    const auto heavier = [](const std::pair<uint64_t, uint32_t> &x, const std::pair<uint64_t, uint32_t> &y) { return x > y; };
    std::make_heap(w.heap.begin(), w.heap.end(), heavier);
    for (uint32_t node = n_leaf; node < n_node; ++node) {
        uint64_t sum = 0;
        for (int child = 0; child < 2; ++child) {
            std::pop_heap(w.heap.begin(), w.heap.end(), heavier);
            sum += w.heap.back().first;
            w.up[w.heap.back().second] = node;
            w.heap.pop_back();
        }
        w.weight[node] = sum;
        w.heap.emplace_back(sum, node);
        std::push_heap(w.heap.begin(), w.heap.end(), heavier);
    }
    w.depth.assign(n_node, 0);
    for (uint32_t v = n_node - 1; v-- > 0;) w.depth[v] = w.depth[w.up[v]] + 1;
    unsigned __int128 bits = 0;
    for (uint32_t i = 0; i < n_leaf; ++i) bits += (unsigned __int128)w.weight[i] * w.depth[i];
    // the root's weight is the number of symbols
    return (double)((long double)bits / (long double)w.weight[n_node - 1]);
}

}  // namespace

extern "C" {

double gg_compression_ratio(double bits, double fixed_length_bits) { return 1.0 - bits / fixed_length_bits; }

gg_status gg_eg_rate(gg_ctx *ctx, const uint64_t *hist, int32_t n_hist, int32_t qmin, int32_t qmax, int32_t k,
                     double *eg_bits, void *stream)
{
    if (!ctx || !hist || !eg_bits || k < 0 || k > 30) return GG_ERR_INVALID_ARG;
    gg_status st = check_hist(0, nullptr, 0, qmin, qmax);
    if (st != GG_OK || n_hist < 0) return GG_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    GG_CUDA(ctx, launch_eg_rate(hist, n_hist, qmax - qmin + 1, qmin, k, eg_bits, static_cast<cudaStream_t>(stream)));
    ctx->launches += n_hist > 0;
    return GG_OK;
}

gg_status gg_eg_rate_grad(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, gg_dtype dtype, const float *step, int32_t k,
                          double lambda, int32_t qmin, int32_t qmax, const gg_seg *grad, gg_dtype grad_dtype,
                          int accumulate, void *stream)
{
    if (!ctx || !grad || (n_seg > 0 && !step) || k < 0 || k > 30 || qmax < qmin) return GG_ERR_INVALID_ARG;
    gg_status st = check_segs(segs, n_seg, dtype);
    if (st != GG_OK) return st;
    st = check_grad(segs, grad, n_seg, grad_dtype);
    if (st != GG_OK) return st;
    if (n_seg == 0) return GG_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    Plan *p = nullptr;
    st = get_plan(ctx, segs, n_seg, dtype, grad, grad_dtype, nullptr, &p, stream);
    if (st != GG_OK) return st;
    GG_CUDA(ctx, launch_eg_grad(p->map, dtype, grad_dtype, step, qmin, qmax, k, lambda, accumulate,
                                static_cast<cudaStream_t>(stream)));
    ctx->launches += p->n_tiles > 0;
    mark_used(p, static_cast<cudaStream_t>(stream));
    return GG_OK;
}

gg_status gg_code_stats(gg_ctx *ctx, const uint64_t *hist, int32_t n_hist, int32_t qmin, int32_t qmax, int32_t k,
                        double *eg_bits, double *hm_bits, double *fl_bits, void *stream)
{
    if (!ctx || !hist || n_hist < 0 || k < 0 || k > 30 || qmax < qmin) return GG_ERR_INVALID_ARG;
    if ((int64_t)qmax - (int64_t)qmin + 1 > (1ll << 24)) return GG_ERR_INVALID_ARG;
    if (n_hist == 0) return GG_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    const int64_t n_bins = (int64_t)qmax - qmin + 1;
    std::vector<uint64_t> host;
    try { host.resize((size_t)n_hist * (size_t)n_bins); } catch (...) { return GG_ERR_NOMEM; }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    GG_CUDA(ctx, cudaMemcpyAsync(host.data(), hist, sizeof(uint64_t) * host.size(), cudaMemcpyDeviceToHost, cs));
    GG_CUDA(ctx, cudaStreamSynchronize(cs));
    HuffmanScratch scratch;
    for (int32_t h = 0; h < n_hist; ++h) {
        const uint64_t *row = host.data() + (size_t)h * (size_t)n_bins;
        // occupied range of the table (first > last: empty)
        int64_t first = 0, last = n_bins - 1;
        while (first <= last && row[first] == 0) ++first;
        while (last >= first && row[last] == 0) --last;
        if (eg_bits) {
            // a k-th order code spends 2 * top_bit(m + 2^k) - k + 1 bits on the unsigned symbol m; the mapping
            // of Eq. 6 interleaves the signs, m = 2|q| - [q > 0]
            unsigned __int128 bits = 0;
            uint64_t symbols = 0;
            for (int64_t b = first; b <= last; ++b) {
                const uint64_t c = row[b];
                if (c == 0) continue;
                const int64_t q = (int64_t)qmin + b;
                const uint64_t m = 2 * (uint64_t)(q < 0 ? -q : q) - (q > 0 ? 1u : 0u);
                bits += (unsigned __int128)c * (uint64_t)(2 * top_bit(m + (1ull << k)) - k + 1);
                symbols += c;
            }
            eg_bits[h] = symbols != 0 ? (double)((long double)bits / (long double)symbols) : 0.0;
        }
        if (hm_bits) hm_bits[h] = huffman_bits(row, n_bins, scratch);
        // a fixed-length code numbers the last - first + 1 symbols of the occupied range
        if (fl_bits) fl_bits[h] = last > first ? (double)(top_bit((uint64_t)(last - first)) + 1) : 0.0;
    }
    return GG_OK;
}

gg_status gg_gct_step(gg_ctx *ctx, const gg_seg *g, int32_t n_seg, gg_dtype g_dtype, const gg_seg *ghat, const gg_seg *w,
                      const float *step, int32_t k, int32_t qmin, int32_t qmax, double eta, double lambda, double eps,
                      int64_t t, void *stream)
{
    if (!ctx || !ghat || !w || (n_seg > 0 && !step) || k < 0 || k > 30 || qmax < qmin || !(eta > 0.0)) return GG_ERR_INVALID_ARG;
    gg_status st = check_segs(g, n_seg, g_dtype);
    if (st != GG_OK) return st;
    st = check_grad(g, ghat, n_seg, GG_F32);
    if (st != GG_OK) return st;
    st = check_grad(g, w, n_seg, GG_F32);
    if (st != GG_OK) return st;
    if (n_seg == 0) return GG_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return GG_ERR_CUDA;
    Plan *pg = nullptr, *pw = nullptr;
    st = get_plan(ctx, g, n_seg, g_dtype, ghat, GG_F32, nullptr, &pg, stream);
    if (st != GG_OK) return st;
    st = get_plan(ctx, w, n_seg, GG_F32, nullptr, 0, nullptr, &pw, stream);      // (for its device table of the weight addresses)
    if (st != GG_OK) return st;
    GG_CUDA(ctx, launch_gct_step(pg->map, const_cast<void *const *>(reinterpret_cast<const void *const *>(pw->map.seg_ptr)),
                                 g_dtype, step, qmin, qmax, k, eta, lambda, eps, t >= 2 ? 1 : 0,
                                 static_cast<cudaStream_t>(stream)));
    ctx->launches += pg->n_tiles > 0;
    mark_used(pg, static_cast<cudaStream_t>(stream));
    mark_used(pw, static_cast<cudaStream_t>(stream));
    return GG_OK;
}

}  // extern "C"
