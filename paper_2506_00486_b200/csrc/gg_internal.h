// Internal declarations shared by the translation units of the library (not installed).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gg.h"

namespace gg {

// Elements per tile.  A tile never crosses a segment; a segment of len elements has
// ceil(len / kTile) tiles and the last one may be ragged.
constexpr int kTile = 16384;
constexpr int kStreamThreads = 256;
// Shared-memory histogram window: symbols [-kWindow/2, kWindow/2) are counted on chip, the
// (rare) rest goes straight to global memory.
constexpr int kWindow = 4096;

enum StreamFlags : int { kMoments = 1, kGrad = 2, kHist = 4 };

// Device-side view of a plan: where each tile lives.
struct TileMap {
    const void *const *seg_ptr;   // [n_seg] input segments
    void *const *grad_ptr;        // [n_seg] gradient segments (may be null)
    const int64_t *seg_len;       // [n_seg]
    const int32_t *tile_prefix;   // [n_seg + 1] first tile of each segment
    const int32_t *tile_seg;      // [n_tiles] owning segment of each tile
    const int32_t *hist_id;       // [n_seg] (null: the segment index)
    int32_t n_seg;
    int32_t n_tiles;
};

// Per-tile partial results (fixed-order reduction happens in the per-segment kernels).
struct TileScratch {
    double *s1;       // sum |x|
    double *s2;       // sum x^2
    double *pen;      // sum |x| |g|   (penalty = that / beta)
    uint32_t *bad;    // non-finite entries
    float *xmin;      // smallest and largest entry (NaN ignored): decide whether a symbol clamps
    float *xmax;
};

struct StreamArgs {
    TileMap map;
    TileScratch part;
    // gradient
    const double *beta;
    const double *alpha;
    double lambda;
    int mean_reduction;
    int accumulate;
    // histogram
    const float *step;
    int32_t qmin, qmax;
    uint64_t *hist;
    uint64_t *clamped;   // [2 * n_hist] or null
};

struct FitArgs {
    TileMap map;
    TileScratch part;
    double *beta, *alpha, *sum_abs, *sum_sq;
    int64_t *count;
    uint32_t *flags;
    const double *seed;       // the fit table (launch_fit_seed_table), or null: search with lgamma evaluations
    int step_from_alpha;
    double step_scale;
    float *step_out;
    // when a histogram is part of the call: GG_FLAG_CLAMPED_SYMBOLS from the segment's extremes
    int hist_on;
    const float *step;
    int32_t qmin, qmax;
};

cudaError_t launch_stream(int flags, gg_dtype in_dtype, gg_dtype grad_dtype, bool has_grad_out,
                          const StreamArgs &a, cudaStream_t st);
// bf16-input sweeps with a gradient and/or a histogram: persistent CTAs, table look-up gradient,
// histogram over bf16 bit patterns.  sm_count sizes the grid.
cudaError_t launch_tail_bf16(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a,
                             int sm_count, cudaStream_t st);
// Whole pass for short bf16 segments: one warp per segment does the moments, the fit, the gradient
// and the histogram while the segment is still in cache, so DRAM sees one read and one write.
constexpr int kSmallSegMax = 16384;   // longest segment the kernel takes (elements)
constexpr int kSeedCells = 2048;      // cells of the ln(beta) grid that seeds the moment-ratio inversion
struct SmallArgs {
    TileMap map;                       // seg_ptr, grad_ptr, seg_len, hist_id, n_seg are used
    double *beta, *alpha, *sum_abs, *sum_sq;
    int64_t *count;
    uint32_t *flags;
    double *penalty;                   // may be null
    double lambda;
    int mean_reduction, accumulate;
    int do_grad;                       // gradient and penalty wanted
    int do_hist;
    const float *step;                 // given steps (null with step_from_alpha)
    int step_from_alpha;
    double step_scale;
    float *step_out;
    int32_t qmin, qmax;
    uint64_t *hist;
    uint64_t *clamped;
    const double *seed;                // the fit table (launch_fit_seed_table)
    uint32_t *cta_counts;              // scratch, kSmallSlotWords words per CTA (small_grid CTAs); needed with do_hist
};
constexpr int kSmallSlotWords = 8200;  // a CTA's count cells and its histogram key
int small_grid(int32_t n_seg, int sm_count);   // CTAs launch_small_bf16 uses
cudaError_t launch_small_bf16(gg_dtype grad_dtype, const SmallArgs &a, int sm_count, cudaStream_t st);
// Fills the fit table, 2 * (kSeedCells + 1) doubles: ln rho(beta_i) and then ln(alpha/sigma)(beta_i), ln beta_i
// evenly spaced over [ln GG_BETA_LO, ln GG_BETA_HI].
cudaError_t launch_fit_seed_table(double *table, cudaStream_t st);

// fp32-input sweeps with a gradient and/or a histogram but no moments (flags in kGrad, kHist, kGrad | kHist):
// persistent CTAs, table + series gradient, symbol counts in shared memory.
cudaError_t launch_tail_f32(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a, int sm_count,
                            cudaStream_t st);
cudaError_t launch_fit(const FitArgs &a, cudaStream_t st);
cudaError_t launch_penalty_finalize(const TileMap &map, const TileScratch &part, const double *beta,
                                    double *penalty, cudaStream_t st);
// scratch: 2 * kEntSplit * n_hist doubles
constexpr int kEntSplit = 16;
cudaError_t launch_entropy(const uint64_t *hist, int32_t n_hist, int32_t n_bins, double *entropy_bits,
                           double *scratch, cudaStream_t st);
cudaError_t launch_eg_rate(const uint64_t *hist, int32_t n_hist, int32_t n_bins, int32_t qmin, int32_t k, double *eg_bits,
                           cudaStream_t st);
cudaError_t launch_eg_grad(const TileMap &map, gg_dtype in_dtype, gg_dtype grad_dtype, const float *step, int32_t qmin,
                           int32_t qmax, int32_t k, double lambda, int accumulate, cudaStream_t st);
// map: the gradient segments with the stored equivalent gradients (fp32) as grad_ptr; w_ptr: the weights (fp32)
cudaError_t launch_gct_step(const TileMap &map, void *const *w_ptr, gg_dtype g_dtype, const float *step, int32_t qmin,
                            int32_t qmax, int32_t k, double eta, double lambda, double eps, int apply_h, cudaStream_t st);
cudaError_t launch_sample(const TileMap &map, gg_dtype dtype, const double *beta, const double *alpha,
                          uint64_t seed, uint32_t tensor_id0, uint32_t *max_attempts, cudaStream_t st);

}  // namespace gg
