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

// kEg (with kGrad and kHist): the gradient is that of lambda * R, R the mean Exponential-Golomb code length of the
// quantised symbols (Eq. 6-7), instead of that of the GG penalty
enum StreamFlags : int { kMoments = 1, kGrad = 2, kHist = 4, kEg = 8 };

// Moments are summed in fp32 over a short run of elements and then added in fp64.  The fp32 sums m1 = sum |x|
// and m2 = sum x^2 of a run can stand for the exact ones unless a square left the fp32 range: upwards
// (m2 is inf or nan; an inf or nan entry ends here too) or downwards, into the subnormals (then m2 is tiny;
// a run of zeros is the harmless case of that).  Runs that fail the test are summed again in fp64.
__device__ __forceinline__ bool run_sums_exact_enough(float m1, float m2)
{
    return m2 <= 3.402823466e+38f && (m2 >= 1e-30f || m1 == 0.0f);
}

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
    // standard deviation of every segment when the caller knows it (the fit of the same call wrote it), else null:
    // it places the count windows; without it the sweeps take the scale from a sample of each run
    const double *seg_sd;
    // memory the moments sweep of a fused call clears on its way (the histograms of the sweep that follows), so
    // that no separate memset sits between two launches: 16-byte vectors, or null
    uint4 *zero_ptr;
    int64_t zero_vecs;
    int32_t eg_k;        // order of the Exponential-Golomb code (kEg)
};

struct FitArgs {
    TileMap map;
    TileScratch part;
    double *beta, *alpha, *sum_abs, *sum_sq;
    int64_t *count;
    uint32_t *flags;
    const double *seed;       // the fit table (launch_fit_seed_table), or null: search with lgamma evaluations
    double *sd_out;           // [n_seg] or null: sqrt(sum_sq / count) of every segment, for the sweep that follows
    int step_from_alpha;
    double step_scale;
    float *step_out;
    int in_dtype_plus1;       // element type of the segments + 1 (gg_dtype), or 0 when the fit cannot read them again
    // when a histogram is part of the call: GG_FLAG_CLAMPED_SYMBOLS from the segment's extremes
    int hist_on;
    const float *step;
    int32_t qmin, qmax;
};

// Arguments of the one-launch fitted pass that keeps tensors in L2 between their two reads (gg_tail_bf16.cu).
struct ResidentArgs {
    const int4 *groups;      // [n_groups] {first tile, end tile, first segment, end segment} of consecutive segments
    int32_t n_groups;
    uint32_t *arrive;        // [n_groups] streamers that have finished the moments of a group; zero before the launch
    uint32_t *ready;         // [n_groups] 1 once the group's fit is published; zero before the launch
    uint32_t expect;         // arrivals that complete a group (the number of streamers)
    uint32_t wait_cap;       // polls after which a wait gives up
    uint32_t keep_tiles;     // tiles of a group that are read with the evict-last hint (what L2 can hold through the pass)
    FitArgs fit;
};
// grid: CTAs of the launch (streamers + one fitter), at most what resident_bf16_max_grid reports
cudaError_t launch_resident_bf16(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a,
                                 const ResidentArgs &r, int grid, cudaStream_t st);
cudaError_t resident_bf16_max_grid(int flags, gg_dtype grad_dtype, bool has_grad_out, int sm_count, int *max_grid);

// The fitted pass with one thread-block cluster per segment, the segment staged in the cluster's shared memory
// (bf16 input, segments up to cluster_size * cluster_tiles_per_cta() tiles, 16-byte aligned; gg_tail_bf16.cu).
struct ClusterArgs {
    FitArgs fit;
    uint32_t wait_cap;       // polls after which the wait for the bulk copies gives up
    uint32_t extra_tx;       // test hook: bytes the barrier expects beyond what is copied (the wait then runs out)
};
int cluster_tiles_per_cta();
cudaError_t launch_cluster_bf16(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a, const ClusterArgs &c,
                                int cluster_size, int n_clusters, cudaStream_t st);
// clusters of this size that can be resident at once
cudaError_t cluster_bf16_max_clusters(int flags, gg_dtype grad_dtype, bool has_grad_out, int cluster_size, int *max_clusters);

cudaError_t launch_stream(int flags, gg_dtype in_dtype, gg_dtype grad_dtype, bool has_grad_out,
                          const StreamArgs &a, cudaStream_t st);
// The moments sweep for bf16 input by persistent CTAs (the one-CTA-per-tile kernel of launch_stream gives the
// same sums tile by tile).  sm_count sizes the grid.
cudaError_t launch_moments_bf16_sweep(const StreamArgs &a, int sm_count, cudaStream_t st);
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
// Turns the pattern-count slots of n_slots CTAs (kSmallSlotWords words each, key in the last four) into symbols.
cudaError_t launch_small_flush(const uint32_t *cta_counts, int n_slots, int32_t qmin, int32_t qmax, uint64_t *hist, uint64_t *clamped,
                               cudaStream_t st);
cudaError_t launch_small_bf16(gg_dtype grad_dtype, const SmallArgs &a, int sm_count, cudaStream_t st);
// Whole pass for short fp32 segments: one team of four warps per segment, the segment held in registers between the
// moments and the gradient (gg_team.cu).  cta_counts as for launch_small_bf16.
int team_grid(int32_t n_seg, int sm_count);    // CTAs launch_team_f32 uses
cudaError_t launch_team_f32(gg_dtype grad_dtype, const SmallArgs &a, int sm_count, cudaStream_t st);
// Fills the fit table, 2 * (kSeedCells + 1) doubles: ln rho(beta_i) and then ln(alpha/sigma)(beta_i), ln beta_i
// evenly spaced over [ln GG_BETA_LO, ln GG_BETA_HI].
cudaError_t launch_fit_seed_table(double *table, cudaStream_t st);

// fp32-input sweeps with a gradient and/or a histogram, with or without the moments (any flags with kGrad or kHist):
// persistent CTAs, table + series gradient, symbol counts in shared memory.
cudaError_t launch_tail_f32(int flags, gg_dtype grad_dtype, bool has_grad_out, const StreamArgs &a, int sm_count,
                            cudaStream_t st);
// Column segments of a row-major bf16 matrix (gg_fused_channels).  Scratch arrays are indexed
// [row block][column]; the moments kernel and the second kernel cut the rows differently.
constexpr int kChanStrip = 64;        // bf16 columns per strip: 128 contiguous bytes of a row
constexpr int kChanStripF32 = 32;     // fp32 columns per strip: the same 128 bytes
constexpr int kChanMomRows = 512;
constexpr int kChanTabFloats = 2 * 65 * 32 + 2 * 128 * 32;   // A (64 exponents + marker row) and B (128 mantissas), two columns per lane     // rows per CTA of the moments kernel
struct ChanArgs {
    const uint16_t *x;                 // (fp32 kernels read it as float)
    int in_f32;                        // the elements are fp32 (ld counts elements of that type)
    int64_t rows, cols, ld;
    void *grad;                        // may be null
    int64_t grad_ld;
    int accumulate;
    int32_t n_mom_blocks;              // ceil(rows / kChanMomRows)
    int32_t n_slices;                  // row slices per strip in the second kernel
    double *s1, *s2;                   // [n_mom_blocks * cols] partial sums
    uint32_t *bad;
    float *xmin, *xmax;
    double *L, *b;                     // [cols]: |g| = 2^(L + b log2|x|); L is NaN for a column without gradient
    float *amax;                       // [cols] largest finite magnitude
    float *sd;                         // [cols] standard deviation
    double *pen;                       // [n_slices * cols] partial sums of |x| |g|
    float *tab;                        // [strips * kChanTabFloats] gradient tables of every strip
    int32_t *tab_elo;                  // [strips] exponent field of the first row of a strip's A table
    double *beta, *alpha, *sum_abs, *sum_sq;
    int64_t *count;
    uint32_t *flags;
    double *penalty;                   // may be null
    const double *seed;                // the fit table
    double lambda;                     // already divided by rows for GG_MEAN
    int do_grad, do_hist;
    float step;
    int32_t qmin, qmax;
    uint64_t *hist;
    uint64_t *clamped;                 // [2] or null
};
cudaError_t launch_chan_moments(const ChanArgs &a, cudaStream_t st);
cudaError_t launch_chan_fit(const ChanArgs &a, cudaStream_t st);
int chan_slices(int64_t rows, int64_t cols, int sm_count, int strip);      // n_slices the second kernel should use (strip: its columns per strip)
// fp32 input: one column per lane (gg_channels_f32.cu); fit and penalty kernels are those of the bf16 path
cudaError_t launch_chan_moments_f32(const ChanArgs &a, cudaStream_t st);
cudaError_t launch_chan_tail_f32(gg_dtype grad_dtype, const ChanArgs &a, int sm_count, cudaStream_t st);
cudaError_t launch_chan_tail(gg_dtype grad_dtype, const ChanArgs &a, int sm_count, cudaStream_t st);
cudaError_t launch_chan_penalty(const ChanArgs &a, cudaStream_t st);
cudaError_t launch_fit(const FitArgs &a, cudaStream_t st);
cudaError_t launch_penalty_finalize(const TileMap &map, const TileScratch &part, const double *beta,
                                    double *penalty, cudaStream_t st);
// scratch: 2 * kEntSplit * n_hist doubles
constexpr int kEntSplit = 16;
// The entropy of n_hist count tables and / or the penalty sums of n_pen segments in one launch.  scratch: 2 * kEntSplit
// doubles per histogram; done: one counter per histogram, zero between calls (the kernel leaves them so).
cudaError_t launch_finish(const TileMap &map, const TileScratch &part, const double *beta, double *penalty, int32_t n_pen,
                          const uint64_t *hist, int32_t n_hist, int32_t n_bins, double *entropy_bits, double *scratch,
                          uint32_t *done, cudaStream_t st);
cudaError_t launch_entropy(const uint64_t *hist, int32_t n_hist, int32_t n_bins, double *entropy_bits,
                           double *scratch, uint32_t *done, cudaStream_t st);
// penalty[s] = lambda * eg_bits[hist_id[s]] (hist_id: device array)
cudaError_t launch_eg_penalty(const double *eg_bits, const int32_t *hist_id, double lambda, double *penalty, int32_t n_seg,
                              cudaStream_t st);
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
