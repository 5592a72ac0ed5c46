/*
 * gg.h -- C interface of the B200 (sm_100a) generalized-Gaussian (GG) pass.
 *
 * The library runs, per tensor or per segment of a tensor, the data-parallel pass that the
 * GG-prior training framework repeats over weights, activations and gradients:
 *
 *   moments  ->  fit (shape beta, scale alpha)  ->  penalty + elementwise gradient
 *            ->  quantise, symbol histogram, empirical entropy;   and GG sampling for init.
 *
 * Letters.  The density is the paper's Eq. 1 with location 0,
 *     f(x) = beta / (2 alpha Gamma(1/beta)) * exp(-(|x|/alpha)^beta),
 * where THIS interface writes the shape as beta and the scale as alpha (Eq. 1 prints them as
 * nu and beta).  sigma^2 = alpha^2 Gamma(3/beta)/Gamma(1/beta) (Eq. 2-3).
 *
 * Conventions.
 *  - Every function returns a gg_status; nothing throws, aborts or prints.
 *  - "device" pointers are CUDA global memory of the context's device; "host" pointers are
 *    ordinary process memory.  The caller owns every buffer it passes; the library keeps no
 *    caller pointer beyond the work it has enqueued.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only
 *    enqueue work; they do not wait for the device.  Exception: the first call that sees a new
 *    segment layout (lengths, dtype, histogram ids, and the addresses) allocates and uploads a
 *    small plan with blocking calls; make that first call outside stream capture.  A context
 *    keeps up to 64 plans, up to 16 of them for one layout at different addresses.  When the
 *    same layout comes with addresses no plan has (buffers that an allocator moved, the same
 *    shapes in another layer) and the layout has its 16 plans or the context its 64, the least
 *    recently used plan of that layout is pointed at the new addresses: two small uploads from
 *    pinned memory, ordered on `stream`, no allocation and no wait for the device (also outside
 *    stream capture: a replayed upload would carry the addresses of capture time).  Only a new
 *    layout in a full context frees the oldest plan, after waiting for the work last enqueued
 *    with it (an event; the whole device if that work was captured in a graph); and a call that
 *    needs more histogram or channel scratch than any before it reallocates that scratch after
 *    waiting for the device.  A context serves one stream at a time.
 *  - A segment is a contiguous run of `len` elements.  Pointers need only element alignment;
 *    16-byte aligned segments take the vectorised path.  Long segments stream fastest when input
 *    and gradient sit at the same element offset from a 1 KB boundary (slices of aligned buffers
 *    do): the kernels then start their vector body where both begin a block.  Unrelated offsets
 *    of the two measured up to 6 % slower on the 7B-sized sweep.
 *  - Per-segment conditions are reported in `flags` (GG_FLAG_*), never as an error status.
 */
#ifndef GG_B200_H
#define GG_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gg_ctx gg_ctx;
typedef int gg_status;

enum {
    GG_OK = 0,
    GG_ERR_INVALID_ARG = 1,   /* null pointer, negative size, inconsistent arguments          */
    GG_ERR_DTYPE = 2,         /* dtype is not GG_F32 / GG_BF16                                 */
    GG_ERR_ALIGNMENT = 3,     /* a pointer is not aligned to its element size                  */
    GG_ERR_WORKSPACE = 4,     /* a fixed-capacity scratch area is too small for the request    */
    GG_ERR_ARCH = 5,          /* the device is not compute capability 10.x                     */
    GG_ERR_CUDA = 6,          /* a CUDA call failed; see gg_last_cuda_error                    */
    GG_ERR_UNIMPLEMENTED = 7,
    GG_ERR_NOMEM = 8          /* a host or device allocation failed                            */
};

typedef enum { GG_F32 = 0, GG_BF16 = 1 } gg_dtype;

/* One contiguous segment.  `ptr` is device memory (host memory for gg_fused_host). */
typedef struct {
    void   *ptr;
    int64_t len;
} gg_seg;

/* Per-segment flag bits written by gg_fit / gg_fused. */
#define GG_FLAG_DEGENERATE      1u   /* len == 0 or all entries zero: beta = alpha = 0       */
#define GG_FLAG_BETA_CLAMPED_LO 2u   /* moment ratio below rho(GG_BETA_LO): beta = GG_BETA_LO */
#define GG_FLAG_BETA_CLAMPED_HI 4u   /* moment ratio above rho(GG_BETA_HI): beta = GG_BETA_HI */
#define GG_FLAG_NONFINITE       8u   /* an entry was inf or nan (left out of the moments)     */
#define GG_FLAG_CLAMPED_SYMBOLS 16u  /* a quantised symbol fell outside [qmin, qmax]          */
#define GG_FLAG_TIMEOUT         32u  /* a bounded wait inside the one-launch fitted pass ran out: no
                                        result of this segment is valid (the context stays usable) */

#define GG_BETA_LO 0.05
#define GG_BETA_HI 20.0

#define GG_SUM  0   /* penalty = lambda * sum_i (|x_i|/alpha)^beta        */
#define GG_MEAN 1   /* the same with lambda replaced by lambda / len      */

#define GG_PARAMS_FITTED 0   /* penalty uses the (beta, alpha) fitted by this call: two reads of x */
#define GG_PARAMS_GIVEN  1   /* penalty uses caller-supplied (beta, alpha); the fit of this call is
                                still produced: one read of x                                    */
#define GG_RATE_EG       2   /* no GG penalty: `grad` gets the gradient of lambda * R, R the mean
                                Exponential-Golomb code length of order eg_k of the quantised symbols
                                (Eq. 6-7, in the relaxed form of the gradient constrained training
                                section, as gg_eg_rate_grad computes it), and penalty[s] = lambda * R of
                                the histogram segment s counts into; the fit of this call is still
                                produced: one read of x for moments, gradient and histogram.  Needs a
                                histogram (hist != NULL) with GG_STEP_GIVEN.  gg_fused only           */
#define GG_STEP_GIVEN      0 /* quantiser step[s] supplied by the caller                        */
#define GG_STEP_FROM_ALPHA 1 /* step[s] = (float)(fitted alpha[s] * step_scale), also written out */

/* ---- context ----------------------------------------------------------------------------- */

/* Creates a context on CUDA device `device` (which must be compute capability 10.x).  The
 * context owns plan tables and per-tile scratch, grown on demand and freed by gg_destroy. */
gg_status gg_create(gg_ctx **out, int device);
gg_status gg_destroy(gg_ctx *ctx);

const char *gg_status_str(gg_status s);
int gg_version(void);
/* Text of the last CUDA error seen by this context ("" if none).  Valid until the next call. */
const char *gg_last_cuda_error(const gg_ctx *ctx);
/* Number of kernels this context has launched since creation (for launch accounting). */
int64_t gg_launch_count(const gg_ctx *ctx);
/* Plans this context has built (what = 0: each one an allocation and a blocking upload) and plans it has pointed
 * at other addresses (what = 1) since creation; -1 for any other `what`. */
int64_t gg_plan_stats(const gg_ctx *ctx, int32_t what);

/* ---- host helpers (no device work) --------------------------------------------------------- */

/* Scale for a wanted standard deviation, Eq. 2: alpha = sigma sqrt(Gamma(1/beta)/Gamma(3/beta)). */
double gg_alpha_from_std(double sigma, double beta);
/* Scale of the GG initialisation rule for a d_in x d_out linear layer, Eq. 4-5:
 * sqrt(xi/d_in * Gamma(1/beta)/Gamma(3/beta)); xi = 1 (no activation / sigmoid), 2 (ReLU),
 * 2/(1+k^2) (leaky ReLU with negative slope k).  beta = 2, xi = 2 is He initialisation. */
double gg_init_alpha(int64_t d_in, double xi, double beta);
/* Differential entropy of Eq. 1 in bits: (1/beta + ln(2 alpha Gamma(1/beta)/beta)) / ln 2. */
double gg_diff_entropy_bits(double alpha, double beta);

/* ---- the steps ------------------------------------------------------------------------------ */

/* Moments and fit of each segment (the "fitted with GGD" step behind the paper's Fig. 1; the
 * method is the moment-ratio inversion
 *     (E|x|)^2 / E[x^2] = Gamma(2/beta)^2 / (Gamma(1/beta) Gamma(3/beta)),
 * which has one root because the right side increases with beta; then alpha from Eq. 2 with
 * sigma^2 = sum_sq / count).
 *   segs      host array of n_seg segments (device data of type `dtype`)
 *   beta, alpha, sum_abs, sum_sq   device double[n_seg], outputs (sum_abs, sum_sq may be NULL)
 *   count     device int64[n_seg] output (= len; may be NULL)
 *   flags     device uint32[n_seg] output (may be NULL)
 * beta is clamped to [GG_BETA_LO, GG_BETA_HI]; a degenerate segment gives beta = alpha = 0. */
gg_status gg_fit(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, gg_dtype dtype,
                 double *beta, double *alpha, double *sum_abs, double *sum_sq,
                 int64_t *count, uint32_t *flags, void *stream);

/* GG distribution penalty and its gradient for given per-segment parameters (the rate term of the
 * rate-distortion objective J = D + lambda R, with R the GG negative log-likelihood without its
 * constants):
 *     penalty[s] = lambda_s * sum_i (|x_i|/alpha_s)^beta_s
 *     g_i        = lambda_s * beta_s * sign(x_i) * |x_i|^(beta_s - 1) / alpha_s^beta_s,  g = 0 at x = 0
 * with lambda_s = lambda (GG_SUM) or lambda/len_s (GG_MEAN).  beta, alpha are constants with
 * respect to x.  beta_s <= 0 or alpha_s <= 0 (a degenerate fit) gives zeros.
 *   beta, alpha   device double[n_seg], inputs
 *   grad          host array of n_seg segments (device data of grad_dtype); grad[s].len must equal
 *                 segs[s].len; NULL = penalty only
 *   accumulate    0: grad = g;  1: grad += g
 *   penalty       device double[n_seg] output (may be NULL) */
gg_status gg_penalty_grad(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, gg_dtype in_dtype,
                          const double *beta, const double *alpha, double lambda, int reduction,
                          const gg_seg *grad, gg_dtype grad_dtype, int accumulate,
                          double *penalty, void *stream);

/* Quantised-symbol histogram and empirical entropy, the rate measure.  The quantiser is the
 * paper's floor quantiser (the forward value of STE(x) = x - sg(x - floor(x)) applied to x/step),
 * with the scaling defined in fp32 so that every symbol is unique:
 *     inv = (float)(1.0/(double)step[s]);  q_i = clamp(floor(fl32(x_i * inv)), qmin, qmax).
 * NaN entries are skipped.
 *   step        device float[n_seg]
 *   hist_id     host int32[n_seg] or NULL; segment s adds to histogram hist_id[s] (NULL: s itself,
 *               which requires n_hist == n_seg)
 *   hist        device uint64[n_hist * (qmax-qmin+1)]; zeroed first unless accumulate != 0
 *   entropy_bits  device double[n_hist]: H = log2 N - (1/N) sum_{c>0} c log2 c (may be NULL)
 *   clamped_lo_hi device uint64[2*n_hist]: symbols moved up to qmin / down to qmax (may be NULL;
 *               zeroed first unless accumulate) */
gg_status gg_rate_hist(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, gg_dtype dtype,
                       const float *step, const int32_t *hist_id, int32_t n_hist,
                       int32_t qmin, int32_t qmax, uint64_t *hist, int accumulate,
                       double *entropy_bits, uint64_t *clamped_lo_hi, void *stream);

/* GG sampling for initialisation ("initialize weights from GGDs", Eq. 4-5).  Element i of segment
 * s is alpha_s * sign * G^(1/beta_s) with G ~ Gamma(1/beta_s, 1) by the Marsaglia-Tsang method
 * (normals by Box-Muller), rounded to nearest-even in `dtype`.  All randomness is Philox4x32-10
 * with counter (i mod 2^32, i div 2^32, attempt, tensor_id0 + s) and key (seed mod 2^32,
 * seed div 2^32); the block with attempt = 0xFFFFFFFF gives the sign and the extra uniform
 * of the shape < 1 case.  Any element can therefore be regenerated alone.
 *   out          host array of n_seg segments (device data of `dtype`), outputs
 *   beta, alpha  HOST double[n_seg]
 *   max_attempts device uint32[n_seg] or NULL: largest number of attempts any element needed
 *                (65 = an element exhausted the 64 allowed attempts and was set to 0) */
gg_status gg_sample(gg_ctx *ctx, const gg_seg *out, int32_t n_seg, gg_dtype dtype,
                    const double *beta, const double *alpha, uint64_t seed, uint32_t tensor_id0,
                    uint32_t *max_attempts, void *stream);

/* Arguments of the fused pass.  Pointer meanings are those of the single-step calls above. */
typedef struct {
    const gg_seg *segs;          /* host array [n_seg]                                        */
    int32_t       n_seg;
    int32_t       in_dtype;      /* gg_dtype                                                  */
    /* fit outputs, device [n_seg]; beta and alpha are required                               */
    double   *beta, *alpha, *sum_abs, *sum_sq;
    int64_t  *count;
    uint32_t *flags;
    /* penalty and gradient                                                                   */
    int32_t       param_mode;    /* GG_PARAMS_FITTED, GG_PARAMS_GIVEN or GG_RATE_EG           */
    const double *beta_in, *alpha_in;   /* device [n_seg], GG_PARAMS_GIVEN only               */
    double        lambda;
    int32_t       reduction;     /* GG_SUM or GG_MEAN                                         */
    const gg_seg *grad;          /* host array [n_seg] or NULL                                */
    int32_t       grad_dtype;
    int32_t       accumulate_grad;
    double       *penalty;       /* device [n_seg] or NULL                                    */
    /* quantiser, histogram, entropy                                                          */
    int32_t       step_mode;     /* GG_STEP_GIVEN or GG_STEP_FROM_ALPHA (needs PARAMS_FITTED) */
    const float  *step;          /* device [n_seg], GG_STEP_GIVEN                             */
    double        step_scale;    /* GG_STEP_FROM_ALPHA                                        */
    float        *step_out;      /* device [n_seg], GG_STEP_FROM_ALPHA: the steps used        */
    const int32_t *hist_id;      /* host [n_seg] or NULL                                      */
    int32_t       n_hist, qmin, qmax;
    uint64_t     *hist;          /* device; NULL skips the histogram step                     */
    int32_t       accumulate_hist;
    double       *entropy_bits;  /* device [n_hist] or NULL                                   */
    uint64_t     *clamped_lo_hi; /* device [2*n_hist] or NULL                                 */
    /* GG_RATE_EG only                                                                        */
    int32_t       eg_k;          /* order of the Exponential-Golomb code, 0 .. 30             */
    double       *eg_bits;       /* device [n_hist] or NULL: mean code length per histogram   */
} gg_fused_args;

/* The whole pass over a list of segments in the fewest sweeps of x: moments -> fit ->
 * penalty + gradient + histogram -> entropy, all enqueued on `stream`.
 * GG_PARAMS_FITTED reads x twice (the gradient needs the fit of the whole segment);
 * GG_PARAMS_GIVEN and GG_RATE_EG read x once (moments, gradient and histogram in the same sweep).
 * The first call with a new layout (segment addresses and lengths) builds and caches its plan with
 * blocking allocations; later calls with that layout only enqueue kernels and memsets on `stream`
 * and may be captured in a CUDA graph (the same holds for gg_fused_channels once its scratch is
 * large enough). */
gg_status gg_fused(gg_ctx *ctx, const gg_fused_args *args, void *stream);

/* ---- code lengths: the rate the paper defines (Eq. 6-7) and its reporting metrics ------------- */

/* Average k-th order Exponential-Golomb code length of each histogram, bits per symbol: the rate
 * function R of Eq. 7.  A symbol q is first mapped to an unsigned one (Eq. 6: q < 0 -> -2q,
 * 0 -> 0, q > 0 -> 2q - 1) and an unsigned m costs 2 floor(log2(m + 2^k)) - k + 1 bits.  Exact
 * 64-bit integer arithmetic up to the final division; an empty histogram gives 0.
 *   hist     device uint64[n_hist * (qmax-qmin+1)], bin 0 = symbol qmin (as written by gg_rate_hist)
 *   k        order of the code, 0 <= k <= 30
 *   eg_bits  device double[n_hist] output */
gg_status gg_eg_rate(gg_ctx *ctx, const uint64_t *hist, int32_t n_hist, int32_t qmin, int32_t qmax,
                     int32_t k, double *eg_bits, void *stream);

/* Elementwise gradient of lambda * R (the paper's dR/dG = 2^(n+2)/(N ln 2) Sign(G)/Map(Quant(G)),
 * with 2^n = 1/step, N the element count of the segment, and the denominator taken as
 * Map(q) + 2^k, the derivative of 2 log2(m + 2^k); the printed form omits 2^k and is undefined at
 * m = 0):
 *     g_i = lambda * 4 inv / (N ln 2) * sign(x_i) / (Map(q_i) + 2^k),   g = 0 at x = 0 and at nan
 * with inv and q_i those of the quantiser of gg_rate_hist.
 *   step   device float[n_segs]
 *   grad   host array of n_seg segments (device data of grad_dtype, same lengths), required
 *   accumulate   0: grad = g;  1: grad += g */
gg_status gg_eg_rate_grad(gg_ctx *ctx, const gg_seg *segs, int32_t n_seg, gg_dtype dtype,
                          const float *step, int32_t k, double lambda, int32_t qmin, int32_t qmax,
                          const gg_seg *grad, gg_dtype grad_dtype, int accumulate, void *stream);

/* Reporting metrics of the paper's tables from histograms: Exponential-Golomb, Huffman and
 * fixed-length bits per symbol ("EG", "HM", "FL" of Section 5.1).  HM is the average length of a
 * Huffman code for the counts (0 for fewer than two occupied bins); FL is
 * ceil(log2(largest occupied symbol - smallest + 1)).  The histograms are copied to the host and
 * the call returns after `stream` has finished the work before it: this is a reporting call, not
 * part of a training step.
 *   eg_bits, hm_bits, fl_bits   HOST double[n_hist] outputs (each may be NULL) */
gg_status gg_code_stats(gg_ctx *ctx, const uint64_t *hist, int32_t n_hist, int32_t qmin, int32_t qmax,
                        int32_t k, double *eg_bits, double *hm_bits, double *fl_bits, void *stream);

/* Compression ratio of a variable-length code against the fixed-length one, C = 1 - bits / FL
 * (the C_EG and C_HM columns of the paper's tables). */
double gg_compression_ratio(double bits, double fixed_length_bits);

/* One step of gradient constrained training for a list of tensors, the elementwise lines of
 * Algorithm 2 in one streaming pass (three reads, two writes per element):
 *     h      = ( -(1/eta) g / (ghat + eps) + 1/eta ) * [t >= 2]      (curvature estimate)
 *     ghat  <- g + lambda * dR/dg * h                                 (stored for the next step)
 *     w     <- w - eta * ghat
 * with dR/dg the gradient of gg_eg_rate_grad for lambda = 1.  Arithmetic is fp64, storage fp32.
 *   g      host array of n_seg segments (device data of g_dtype): this step's gradients
 *   ghat   host array of n_seg segments (device float32, same lengths): in: the equivalent gradients
 *          of the previous step (not read when t < 2); out: this step's
 *   w      host array of n_seg segments (device float32, same lengths): the weights, updated in place
 *   step   device float[n_seg]: quantiser steps
 *   t      the training step, 1-based */
gg_status gg_gct_step(gg_ctx *ctx, const gg_seg *g, int32_t n_seg, gg_dtype g_dtype, const gg_seg *ghat,
                      const gg_seg *w, const float *step, int32_t k, int32_t qmin, int32_t qmax,
                      double eta, double lambda, double eps, int64_t t, void *stream);

/* Optional device timing of the sweeps inside gg_fused (no counterpart in the paper: measurement
 * support).  While enabled, gg_fused records a CUDA event pair on the caller's stream around its
 * first sweep (moments, or the single combined sweep of GG_PARAMS_GIVEN) and around its second
 * sweep (gradient + histogram).  gg_timing_read waits for the recorded events, returns the summed
 * milliseconds and the number of launches of each kind since the last read, and forgets them. */
gg_status gg_timing_enable(gg_ctx *ctx, int enable);
gg_status gg_timing_read(gg_ctx *ctx, double *ms_first, int64_t *n_first, double *ms_tail, int64_t *n_tail);

/* The one-launch form of the fitted pass, and its knobs (no counterpart in the paper).  With bf16 input and
 * GG_PARAMS_FITTED, gg_fused can run moments, fit and gradient + histogram of every tensor in ONE cooperative
 * launch: all CTAs walk the tensors together (in groups of about 28 MB), a fitting CTA publishes the parameters
 * of a group once every streaming CTA has delivered its moments, and the second read of the group follows while L2
 * still holds it, so DRAM sees less than two reads of x.  On B200 this form is SLOWER than the two-launch form
 * (the per-group hand-over stalls all CTAs at once, while the two-launch sweeps keep DRAM busy), so it is off
 * unless switched on here.  CTAs of that launch wait for one another (arrival counters and ready words in the
 * plan); every such wait gives up after a fixed number of polls, marks the segments GG_FLAG_TIMEOUT and lets the
 * kernel end, so a wait that cannot be satisfied costs a fraction of a second and leaves the context usable.
 *   GG_HOOK_RESIDENT_MODE   0 (default): two launches; 1: the one-launch form whenever it can run
 *   GG_HOOK_EXTRA_ARRIVALS  arrivals the fitting CTA waits for beyond the CTAs that exist (default 0); a positive
 *                           value makes its wait run out: the way to test the time-out path without any fault (the
 *                           one-cluster-per-segment form then expects 16 bytes per unit more than it copies, with
 *                           the same effect on its wait)
 *   GG_HOOK_WAIT_CAP        polls (about half a microsecond each) after which a wait gives up (default 2^18) */
#define GG_HOOK_RESIDENT_MODE  0
#define GG_HOOK_EXTRA_ARRIVALS 1
#define GG_HOOK_WAIT_CAP       2
#define GG_HOOK_CLUSTER_MODE   3   /* the fitted pass with bf16 segments of 32 KB .. 2 MB staged in the shared memory of a
                                      thread-block cluster, so that DRAM sees x once (6 bytes per element instead of 8):
                                      0 (default) never; 1 when the layout suits (segments of similar length, enough of
                                      them); 2 whenever every segment fits a cluster of 16 and starts on a 16-byte
                                      boundary.  It moves fewer bytes but takes longer than the two sweeps on an idle
                                      B200 (a cluster works through load, fit and tables one after the other), which is
                                      why it is off unless asked for. */
gg_status gg_test_hook(gg_ctx *ctx, int32_t what, int64_t value);

/* Bounds-checking build (no counterpart in the paper: a debugging aid that stands in for a memory checker).  A
 * library built with -DGG_BOUNDS (paper_2506_00486_b200/build.py --bounds) tests the index of every checked global
 * load and store of its streaming kernels against the extent of the segment or buffer it belongs to, counts the
 * ones that would have left it and skips them; nothing traps.  Returns the number of such accesses since the library
 * was loaded (after waiting for the device), or -1 from a normal build, which has no checks. */
int64_t gg_debug_bounds_violations(void);

/* The same pass for data that lives in HOST memory: every pointer of `args` that gg_fused documents
 * as device memory (segment data, fit outputs, gradient segments, step, histogram, entropy, ...) is
 * here a host pointer.  The library stages segments through device buffers of its own in chunks of
 * at most `chunk_bytes` of input (0 = default), overlapping copies with kernels, and returns after
 * all results are in host memory.  Pinned host buffers make the copies asynchronous. */
gg_status gg_fused_host(gg_ctx *ctx, const gg_fused_args *args, int64_t chunk_bytes);

/* ---- channel-wise (strided) segments ------------------------------------------------------------ */

/* Arguments of the fused pass over the COLUMNS of a row-major matrix: segment c is the column
 * x[0 * ld + c], x[1 * ld + c], ..., x[(rows-1) * ld + c] (one GG per channel of an activation or
 * input channel of a weight matrix; rows of a matrix are contiguous segments and go through
 * gg_fused).  The paper fits one GG per tensor; per-channel fits are this library's generalisation
 * of the same pass and every formula is that of gg_fit, gg_penalty_grad and gg_rate_hist.
 * All columns are quantised with one step into ONE histogram (the rate of the whole tensor). */
typedef struct {
    const void *x;               /* device, element (r, c) at x[r * ld + c]                   */
    int64_t     rows, cols, ld;  /* ld >= cols, in elements                                   */
    int32_t     in_dtype;        /* GG_BF16 or GG_F32                                         */
    /* fit outputs, device [cols]; beta and alpha are required                                */
    double   *beta, *alpha, *sum_abs, *sum_sq;
    int64_t  *count;
    uint32_t *flags;
    /* penalty and gradient with the fitted parameters of each column                         */
    double    lambda;
    int32_t   reduction;         /* GG_SUM or GG_MEAN (lambda / rows)                         */
    void     *grad;              /* device matrix of grad_dtype, element (r, c) at            */
    int64_t   grad_ld;           /*   grad[r * grad_ld + c]; NULL: no gradient                */
    int32_t   grad_dtype;
    int32_t   accumulate_grad;
    double   *penalty;           /* device [cols] or NULL                                     */
    /* quantiser, histogram, entropy                                                          */
    float     step;              /* one step for the matrix                                   */
    int32_t   qmin, qmax;
    uint64_t *hist;              /* device [qmax-qmin+1]; NULL skips the histogram step       */
    int32_t   accumulate_hist;
    double   *entropy_bits;      /* device [1] or NULL                                        */
    uint64_t *clamped_lo_hi;     /* device [2] or NULL                                        */
} gg_channel_args;

/* moments -> fit -> penalty + gradient + histogram -> entropy for every column of the matrix, all
 * enqueued on `stream`: the matrix is read twice (row-major, coalesced: a strip of 64 bf16 or 32 fp32
 * columns is 128 contiguous bytes of every row), the second time from L2 when it fits there.  Results per
 * column equal those of gg_fused on the gathered column within the same tolerances; sums over a
 * column are reduced in a fixed order.  GG_FLAG_CLAMPED_SYMBOLS is set per column when a histogram
 * is taken.  The first call with a larger matrix than any before allocates scratch (blocking).
 * Errors: GG_ERR_DTYPE for an unknown dtype, GG_ERR_INVALID_ARG for ld < cols, negative sizes, a missing
 * required pointer, qmin > qmax or a step that is not a positive finite number, GG_ERR_ALIGNMENT for x or
 * grad not element aligned, GG_ERR_WORKSPACE for more than 65535 * 512 rows. */
gg_status gg_fused_channels(gg_ctx *ctx, const gg_channel_args *args, void *stream);

/* Moments and fit of ONE segment without allocating anything (the paper has no counterpart: this is
 * gg_fit for callers that cannot allocate).  gg_fit keeps its tile tables and per-tile partial sums in
 * a plan that the context obtains with cudaMalloc the first time it sees a layout.  Callers that run
 * while an allocator owns or has frozen the device's memory (a caching pool that must not see side
 * allocations, a step whose buffer addresses must not move, a plug-in that is given buffers and a
 * stream and nothing more) cannot afford that.  This call needs no context and calls neither
 * cudaMalloc, cudaFree nor any allocating routine: its tables and partials live in a fixed array of
 * about 0.7 MB inside the library image.  The CUDA runtime places that array, and the code of the three kernels,
 * on a device when the library's module is first loaded there, which by default happens lazily at the first call
 * on that device, and the device then holds them until the process exits.  A caller whose allocator is about to
 * take or freeze all device memory should therefore make one warm-up call per device and element type
 * beforehand (or run with CUDA_MODULE_LOADING=EAGER); a first call made when no memory is left can fail with
 * GG_ERR_CUDA.
 *   device    CUDA device that owns `x` and the outputs (compute capability 10.x, index < 64)
 *   x         device data of type `dtype`, `len` elements, element aligned
 *   len       0 <= len <= gg_fit_noalloc_max_len() (2^28 elements); a longer segment is refused with
 *             GG_ERR_WORKSPACE and nothing is enqueued
 *   beta, alpha, sum_abs, sum_sq, count, flags   device outputs of ONE element each, as in gg_fit
 *             (sum_abs, sum_sq, count, flags may be NULL)
 * The results are those of gg_fit on the same segment up to the rounding of the fp64 partial sums (this call
 * sums tile by tile, gg_fit run by run: the sums agree to about 1e-15 relative).
 * The first call on a device looks up the array's device address and the device's architecture; make
 * that first call before any stream capture begins.  Later calls only enqueue three kernels on
 * `stream`.  All calls on a device share the one array, which keeps the previous call's contents; each
 * call rewrites every entry it reads, so calls that follow one another on the GPU are independent, but
 * two calls whose kernels overlap on the GPU (different streams, no ordering between them) race on
 * the array and give undefined results. */
gg_status gg_fit_noalloc(int device, const void *x, int64_t len, gg_dtype dtype, double *beta,
                         double *alpha, double *sum_abs, double *sum_sq, int64_t *count,
                         uint32_t *flags, void *stream);
int64_t gg_fit_noalloc_max_len(void);

#ifdef __cplusplus
}
#endif
#endif /* GG_B200_H */
