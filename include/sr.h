/*
 * sr.h - C ABI of the B200 (sm_100a) pixel-adaptive dictionary regression library.
 *
 * The library computes the last two stages of a LAPAR-style super-resolution
 * model together with the up-sampling they consume (paper Section II-A,
 * Eq. 2-3): the LR image is up-sampled to U, the k x k patch B_i of U around
 * every HR pixel i is taken, the per-pixel filter F_i = Phi_i D is assembled
 * from the dictionary D (L atoms of k*k taps; L is called D in `sr_dims`) and
 * the pixel's coefficients Phi_i, and y_i = F_i B_i^T.  The filter matrix F and
 * the patch matrix B never reach global memory.
 *
 * Conventions shared by every call
 *   - Every data pointer is a DEVICE pointer; `stream` is a cudaStream_t passed
 *     as void* (NULL = the legacy default stream).  `d` is a HOST pointer.
 *   - Layouts, all contiguous, row-major, innermost index last:
 *       lr        [n][c][h][w]           fp32   LR image
 *       hr / out  [n][c][H][W]           fp32   H = h*scale, W = w*scale (out: binary16 with SR_OUT_F16, uint8 with SR_OUT_U8)
 *       coef      [n][D][H][W]           fp32 or binary16 (SR_F32 / SR_F16); one set per
 *                                        frame, shared by the c channels
 *       dict      [D][k*k]               fp32, tap j = a*k + b (a = row) multiplies
 *                                        U[Y + a - p][X + b - p], p = (k-1)/2 (no flip)
 *       idx       [n][s][H][W]           uint8, rank order (plane 0 = largest magnitude);
 *                                        with SR_IDX_GLOBAL: idx[s]
 *       sel       [n][s][H][W]           coefficient dtype; plane q = coefficient of idx plane q
 *       gamma     [s]                    fp32 (SR_IDX_GLOBAL only)
 *   - Ownership: the caller owns every buffer.  The library allocates nothing
 *     the caller must free and keeps no reference after the call's work has
 *     run.  Calls are asynchronous on `stream` and never synchronise the host;
 *     buffers must stay valid until the stream reaches the kernels.  `out`
 *     must not alias an input.  Because of this a sequence of calls can be
 *     recorded into a CUDA graph and replayed; make one ordinary call of each
 *     kind on the device first (the first launch of a kernel there looks up
 *     the status word and sets the kernel's shared-memory limit).
 *   - Errors: every call returns an sr status.  Validation failures return
 *     before anything is launched and write nothing.  Nothing throws, aborts or
 *     prints.  A device-side wait that ran out of its iteration limit is
 *     reported by sr_device_status (the output of that call is then undefined).
 *   - Alignment: lr, hr/out, dict and gamma 4 bytes; coef/sel their element size
 *     (the tensor-core path additionally needs coef 16-byte aligned and W a
 *     multiple of 8, and for per-pixel idx planes idx 16-byte aligned and W a
 *     multiple of 16; other inputs take the general path).
 *   - Value ranges on the tensor-core path (binary16 coefficients, aligned as above, k <= 7, c <= 4): the fp32
 *     dictionary is held as the sum of two binary16 numbers, so every tap (times gamma, in the global-subset mode)
 *     must satisfy |tap| < 65504; taps below 2^-14 in magnitude keep an absolute precision of 2^-25 instead of 22
 *     significant bits.  Coefficients must be finite: the kernel pads the atom count to a multiple of 16 with
 *     neighbouring staged data times zero dictionary rows, and the in-call selection multiplies dropped
 *     coefficients by zero, so one Inf or NaN coefficient makes the outputs of its 128-pixel row segment
 *     unspecified.  The general path has neither restriction.
 */
#ifndef SR_H_
#define SR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sr_dims {
    int32_t n, c, h, w; /* LR batch, channels, height, width (each >= 1)                 */
    int32_t scale;      /* integer up-scaling factor r in [1, 8]                          */
    int32_t k;          /* atom / patch side, odd, in {1,3,5,7,9}                         */
    int32_t D;          /* number of dictionary atoms (the paper's L), 1..256             */
} sr_dims;

enum { SR_F32 = 0, SR_F16 = 1 }; /* coefficient storage type */

enum {
    SR_CLAMP01 = 1u,      /* clamp the output to [0,1] as the last step                                */
    SR_IDX_GLOBAL = 2u,   /* idx[s] (+ gamma[s]) is one atom subset for every pixel                    */
    SR_COEF_COMPACT = 4u, /* the coefficient argument is [n][s][H][W] (selected values), not [n][D][H][W] */
    SR_UPSAMPLE_BILINEAR = 8u, /* stage 1 interpolates linearly between the two nearest LR samples per axis
                                  (the interpolation Section II-A names) instead of the bicubic kernel        */
    SR_OUT_F16 = 16u,          /* regression calls: `out` is binary16 [n][c][H][W]; the fp32 result is rounded
                                  to nearest as it is stored (halves the output traffic).  2-byte alignment.  */
    SR_OUT_U8 = 32u,           /* regression calls: `out` is uint8 [n][c][H][W], an 8-bit image: the fp32 result
                                  clamped to [0,1] (whether or not SR_CLAMP01 is given), times 255, rounded to
                                  nearest, ties to even (a quarter of the output traffic).  Not together with
                                  SR_OUT_F16.                                                                  */
    SR_LUMA_ONLY = 64u         /* regression calls, c = 3 (R, G, B planes) only: the per-pixel filter is applied to
                                  the luma Y = 0.299 R + 0.587 G + 0.114 B of the up-sampled image and the chroma
                                  differences keep their up-sampled values:  out_ch = U_ch + (F . B_Y - U_Y)  at the
                                  pixel.  The common practice of SR models that predict on the Y channel; the paper
                                  has no such variant.  With fp32 output it is composed of the one-channel
                                  regression of the luma frame (the fast kernels) and two small kernels, using
                                  `out` itself as scratch; with binary16 / 8-bit output it runs on the general
                                  fp32 kernel.                                                                  */
};

enum {
    SR_OK = 0,
    SR_ERR_NULL = 1,        /* a required pointer is NULL                        */
    SR_ERR_SHAPE = 2,       /* a size is out of range (n,c,h,w,D < 1; s < 1 or s > D; total size overflow) */
    SR_ERR_UNSUPPORTED = 3, /* scale not in [1,8]; k even or > 9; D > 256; unknown dtype or flag */
    SR_ERR_ALIGN = 4,       /* a pointer is not aligned to its element size      */
    SR_ERR_CUDA = 5,        /* a CUDA runtime call or launch failed              */
    SR_ERR_TIMEOUT = 6,     /* device status only: a bounded device-side wait expired */
    SR_ERR_TOO_LARGE = 7    /* sr_selection_gram_static: more atoms than its built-in scratch holds */
};

/*
 * Stage 1 alone (Section II-A, the up-sampling that feeds the patch matrix B): hr = bicubic(lr).
 * Keys cubic convolution with a = -0.75, half-pixel centres
 * (src = (X + 1/2)/scale - 1/2), tap indices clamped to the image; the result
 * is not clamped.  d->k and d->D are ignored.
 */
int sr_bicubic_upsample(const float* lr, float* hr, const sr_dims* d, void* stream);

/*
 * Stage 1 alone with the interpolation the paper's text names for stage 1
 * (Section II-A: bilinear): the same half-pixel sample point, linear
 * interpolation between the two nearest LR samples per axis, indices clamped
 * to the image.  lr must be finite (the two outer taps of the shared four-tap
 * window are multiplied by zero).  d->k and d->D are ignored.
 */
int sr_bilinear_upsample(const float* lr, float* hr, const sr_dims* d, void* stream);

/*
 * Stages 1, 3 and 4 with every atom (Eq. 2: y_i = F_i B_i^T with F_i = Phi_i D;
 * image form Eq. 3): out[n][c][Y][X] = sum_j (sum_l coef[n][l][Y][X] * dict[l][j]) * B_c[j],
 * patch positions clamped to the HR image (edge replicate).  fp32 accumulation.
 * flags: any of SR_CLAMP01, SR_UPSAMPLE_BILINEAR, SR_OUT_F16 (`out` then points at binary16 elements).
 */
int sr_dict_regress_dense(const float* lr, const void* coef, int coef_dtype, const float* dict, float* out,
                          const sr_dims* d, uint32_t flags, void* stream);

/*
 * Per-pixel top-s selection (the dictionary selective strategy applied per HR
 * pixel; the paper's Section III-A selects one subset for the whole model,
 * which is the SR_IDX_GLOBAL mode of sr_dict_regress_selected): for every
 * pixel the s atoms with the largest |coef|, ties to the lower atom index,
 * written in rank order.  The ordering key is the coefficient's bit pattern
 * with the sign cleared, so -0/+0 and +x/-x tie.  `sel` may be NULL; otherwise
 * it receives the selected coefficients.  flags must be 0.  d->c, d->k unused.
 */
int sr_dict_select(const void* coef, int coef_dtype, uint8_t* idx, void* sel, const sr_dims* d, int s,
                   uint32_t flags, void* stream);

/*
 * Stages 1, 3 and 4 with s atoms per pixel (Section II-A: computations the
 * dictionary gates are skipped; Section III-A, Eq. 6 and Eq. 9 for the global
 * form): out = sum_j (sum_q w_q * dict[a_q][j]) * B_c[j].
 *   flags = 0:               a_q = idx[n][q][Y][X], w_q = coef[n][a_q][Y][X]
 *                            (idx == NULL: the top-s atoms are chosen inside the call and never stored)
 *   SR_COEF_COMPACT:         w_q = coef_or_sel[n][q][Y][X]  (idx required)
 *   SR_IDX_GLOBAL:           a_q = idx[q], w_q = gamma[q] * coef[n][a_q][Y][X]  (gamma NULL = 1);
 *                            with SR_COEF_COMPACT, w_q = gamma[q] * coef_or_sel[n][q][Y][X]
 * SR_CLAMP01, SR_UPSAMPLE_BILINEAR and SR_OUT_F16 may be added to any of these.
 * With idx == NULL the coefficients must be finite (the selection multiplies dropped ones by zero).
 * Kept coefficients are used unchanged (no renormalisation).  The s indices of a pixel must be distinct (as
 * sr_dict_select writes them); repeated indices give an unspecified value for that pixel.  An idx value >= D
 * is the caller's error: that pixel's value is then undefined, but no
 * out-of-range access is made (the value is clamped to D-1).
 */
int sr_dict_regress_selected(const float* lr, const void* coef_or_sel, int coef_dtype, const uint8_t* idx,
                             const float* gamma, const float* dict, float* out, const sr_dims* d, int s,
                             uint32_t flags, void* stream);

/*
 * Dictionary selection search (Section III-A).  The paper keeps alpha * L of the L atoms: a selecting vector beta
 * enters the filter as F = Phi diag(beta) D (Eq. 5-6), beta is found by LASSO (Eq. 7) with lambda doubled and then
 * bisected until about alpha_t L atoms survive, the coefficient layer is re-fitted on the survivors by least squares
 * (Eq. 9: one re-weight gamma_l per kept atom), and alpha_t is lowered step by step (Algorithm 1).  Fine-tuning the
 * whole network is not part of this library; the re-fit of Eq. 9 is the paper's own fast substitute for it.  The
 * result (atom ids + re-weights) is what sr_dict_regress_selected takes with SR_IDX_GLOBAL.
 *
 * sr_selection_gram: everything the search needs from the images.  With z_l[i,c] = coef[l][i] * (dict[l] . B_{i,c})
 * the response of atom l alone at HR pixel i, channel c, and `target` [n][c][H][W] fp32 the ground-truth HR image:
 *     G[l][m] = sum z_l z_m,   b[l] = sum z_l target,   *hh = sum target^2      (device fp64: G [D][D], b [D], hh [1])
 * summed over the pixels listed in `samples` (device int64 flat [n][H][W] indices, nsamples of them; the paper samples
 * its LASSO features too) or over every pixel when samples == NULL, all c channels of each.  Indices outside the
 * tensor are skipped.  flags: SR_UPSAMPLE_BILINEAR or 0.  fp32 arithmetic per 32 pixels, fp64 accumulation; the result
 * does not depend on the order in which thread blocks run.
 * `scratch` is device memory of at least sr_selection_gram_scratch_bytes(d) bytes, 8-byte aligned; the call
 * overwrites it, and two calls that share it must not overlap.  Returns SR_ERR_SHAPE when it is too small.
 */
size_t sr_selection_gram_scratch_bytes(const sr_dims* d);
int sr_selection_gram(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                      const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, const sr_dims* d,
                      uint32_t flags, void* scratch, size_t scratch_bytes, void* stream);

/*
 * sr_selection_gram for callers that cannot allocate device memory where they need the statistics: a pipeline that
 * sizes every buffer once at start-up and then runs under a fixed memory budget, a plug-in whose host application owns
 * the allocator, a service that keeps cudaMalloc (which synchronises the whole device and can fail late) out of its
 * steady state.  Same inputs, outputs and results as sr_selection_gram, but no `scratch` argument: the per-block fp64
 * partial sums live in a device array that is part of the library, 1 660 928 bytes (32 blocks x (80 x 80 + 80 + 8)
 * doubles) held by every GPU that loads the library until the process exits.  Limit: d->D <= 80 atoms; more returns
 * SR_ERR_TOO_LARGE and launches nothing.  The call allocates nothing and frees nothing.  The first call on a device
 * looks up the array's device address (cudaGetSymbolAddress, with that device current) and sets the kernel's
 * shared-memory limit; make that first call before any stream capture begins.  The array is shared by all calls on a
 * device and keeps the previous call's contents; every block clears its part before use, so back-to-back calls on one
 * stream are fine, but two calls that can overlap on the GPU (different streams or host threads) race on it and give
 * wrong sums.  With 32 blocks instead of two per multiprocessor it is slower than sr_selection_gram on large inputs.
 * A convenience of this library; the paper has no counterpart.
 */
int sr_selection_gram_static(const float* lr, const void* coef, int coef_dtype, const float* dict, const float* target,
                             const int64_t* samples, int64_t nsamples, double* G, double* b, double* hh, const sr_dims* d,
                             uint32_t flags, void* stream);

typedef struct sr_search_opts {
    double alpha;        /* fraction of the atoms to keep in the end, in (0, 1]                                   */
    double delta_alpha;  /* the kept fraction falls by this much per step (alpha_{t+1} = alpha_t - delta_alpha)    */
    double eps;          /* a step accepts || beta ||_0 within eps * D of alpha_t * D                              */
    double lambda0;      /* the small lambda the first step starts from (> 0)                                      */
    double tol;          /* coordinate descent stops when no coefficient moved by more than tol in a sweep         */
    int32_t max_sweeps;  /* ... or after this many sweeps                                                          */
    int32_t max_bisect;  /* halvings of the lambda bracket per step                                                */
    int32_t max_steps;   /* rows of `trace`; the search stops after this many steps                                */
} sr_search_opts;

/*
 * sr_selection_search: Algorithm 1 on the Gram statistics (device pointers G [D][D], b [D], hh [1] in fp64, as
 * sr_selection_gram writes them; nrows = number of (pixel, channel) rows they were summed over: the 1/N of Eq. 7),
 * D <= 128.  Writes, all on the device: idx_out [D] the kept atoms in ascending order, gamma_out [D] their re-weights
 * (product over all steps), *count_out how many were kept (-1 when a re-fit met a singular matrix), and per step
 * trace[t][0..5] = alpha_t, lambda used, atoms kept, loss after the beta step, loss after the re-fit, LASSO solves
 * (trace and steps_out may be NULL).  The printed listing's bisection is read as a bisection inside the last doubling
 * step with the feasible solution that keeps the most atoms taken when no lambda lands in the band.
 * `scratch`: device memory of at least sr_selection_search_scratch_bytes(D) bytes, 8-byte aligned.  fp64 throughout;
 * one warp, every sum in a fixed order: the same inputs give the same bits on every run.
 */
size_t sr_selection_search_scratch_bytes(int32_t D);
int sr_selection_search(const double* G, const double* b, const double* hh, double nrows, int32_t D,
                        const sr_search_opts* opts, uint8_t* idx_out, float* gamma_out, int32_t* count_out, double* trace,
                        int32_t* steps_out, void* scratch, size_t scratch_bytes, void* stream);

/* Text for a status code (static storage, never NULL). */
const char* sr_status_string(int status);

/*
 * Synchronises `stream`, then reads and clears the device status word of the
 * current device into *out_status (SR_OK or SR_ERR_TIMEOUT).  Returns SR_OK,
 * SR_ERR_NULL or SR_ERR_CUDA.
 */
int sr_device_status(void* stream, int* out_status);

/*
 * Tile-shape search (Section III-B, restated for this library).  The paper prunes the space of thread-block shapes
 * of its filtering kernel with resource constraints (Eq. 11-12) and searches the rest by measured latency.  Here the
 * tunable shape of a regression launch is: which kernel takes it (first or second tensor-core layout, the FMA-pipe
 * subset kernel, the FMA-pipe gather kernel for index + value planes), the tile height, and the rows per pipeline step; the legal set follows from the shared memory per
 * thread block, the tensor-memory columns and the stage count, and is small enough to time exhaustively.
 * sr_tune_dense / sr_tune_selected take the arguments of the call they tune plus `reps`, run every legal shape
 * (one warm-up launch, then `reps` timed launches between two CUDA events) on the caller's own buffers, and record the
 * fastest for this problem shape (n, c, h, w, scale, k, D, s, flags, coefficient type); later calls of
 * sr_dict_regress_dense / sr_dict_regress_selected with the same shape use it.  They synchronise `stream`, overwrite
 * `out`, and are meant to be called once per shape at start-up; inputs that are not larger than the L2 cache are timed
 * warm.  The per-pixel arithmetic does not depend on the tile shape, so results for one kernel are the same bits for
 * every shape.  *result (may be NULL) receives the choice.  sr_tune_reset forgets every recorded shape.
 */
typedef struct sr_tune_result {
    int32_t kernel;        /* 0 general FMA kernel, 1 first tensor-core layout, 2 second tensor-core layout, 3 subset
                              kernel, 4 gather kernel for index + value planes                                         */
    int32_t tile_rows;     /* tile height (kernels 2, 3 and 4; 0 otherwise)                                            */
    int32_t rows_per_step; /* tile rows per pipeline step (kernel 2; 0 otherwise)                                      */
    int32_t candidates;    /* launch shapes that were legal and timed                                                   */
    float best_us;         /* time per launch of the recorded shape                                                     */
    float default_us;      /* time per launch of the shape the host rules pick without tuning                           */
} sr_tune_result;
int sr_tune_dense(const float* lr, const void* coef, int coef_dtype, const float* dict, float* out, const sr_dims* d,
                  uint32_t flags, int reps, void* stream, sr_tune_result* result);
int sr_tune_selected(const float* lr, const void* coef_or_sel, int coef_dtype, const uint8_t* idx, const float* gamma,
                     const float* dict, float* out, const sr_dims* d, int s, uint32_t flags, int reps, void* stream,
                     sr_tune_result* result);
void sr_tune_reset(void);

/*
 * Regression fused with the producer of the coefficients (Section II-A: the coefficient network ends in convolution
 * and pixel-shuffle layers; Eq. 2-3 then use its output).  When that last layer is a plain convolution over an LR
 * feature map followed by a pixel-shuffle by `scale`,
 *     Phi_l(Y, X) = bias[o] + sum_{ci, dy, dx} feat[Y div r + dy - kc/2][X div r + dx - kc/2][ci] * wconv[o][ci][dy][dx],
 *     o = l r^2 + (Y mod r) r + (X mod r)      (positions outside the map read zero),
 * the coefficient tensor need never exist: F_i = Phi_i D is itself one convolution of the feature map with the weights
 * folded with the dictionary.  sr_producer_fold builds those folded weights once per (network, dictionary);
 * sr_producer_regress computes what sr_dict_regress_dense would compute on that Phi (or, after a fold with a subset,
 * what sr_dict_regress_selected with SR_IDX_GLOBAL would), reading feat instead of coefficients.
 *
 *   wconv  [D*scale^2][cin][kc][kc] fp32 (device), bias [D*scale^2] fp32 (device) or NULL
 *   dict   [D][k*k] fp32;  idx[s] / gamma[s] (device): an atom subset and its weights, or NULL / NULL for every atom
 *          (gamma alone NULL: ones)
 *   feat   [n][h][w][cin] binary16, channels last, 16-byte aligned
 *   folded device buffer of sr_producer_folded_bytes(d, cin, kc) bytes, 16-byte aligned, owned by the caller; its
 *          layout is private to the library and depends on d->scale, d->k, cin, kc (not on n, c, h, w, D)
 *   out    [n][c][H][W], 16-byte aligned; fp32, or binary16 / uint8 with SR_OUT_F16 / SR_OUT_U8
 * flags of sr_producer_regress: SR_CLAMP01, SR_UPSAMPLE_BILINEAR, SR_OUT_F16, SR_OUT_U8.
 * Supported: scale 2, 3 or 4, k in {3, 5, 7} (k <= 5 at scale 3), c <= 3, cin = 32, kc in {1, 3}; anything else is SR_ERR_UNSUPPORTED (there
 * is no slower path behind this call) and sr_producer_folded_bytes returns 0.  The folded weights are rounded to
 * binary16 (the bias keeps about 22 bits), feature values must be finite; results agree with the fp64 definition
 * within the binary16 tolerance of the other calls.  Asynchronous on `stream`; device-side waits are bounded as in
 * the other tensor-core calls (sr_device_status).
 */
size_t sr_producer_folded_bytes(const sr_dims* d, int cin, int kc);
int sr_producer_fold(const float* wconv, const float* bias, const float* dict, const uint8_t* idx, const float* gamma,
                     int s, void* folded, size_t folded_bytes, const sr_dims* d, int cin, int kc, void* stream);
int sr_producer_regress(const float* lr, const void* feat, const void* folded, size_t folded_bytes, float* out,
                        const sr_dims* d, int cin, int kc, uint32_t flags, void* stream);

/*
 * Sustained issue rate of an arithmetic pipe of the current device, for the roofline of the kernels that are bound by
 * one (the selection networks by integer max/min, the general and subset regressions by fp32 multiply-add):
 * kind 0 = integer max/min, kind 1 = fp32 multiply-add, kind 2 = packed fp32 multiply-add (fma.rn.f32x2, counted as two
 * multiply-adds per lane and instruction).  Runs a register-only kernel a few times on `stream`,
 * synchronises it, and writes lane operations per second to *lane_ops_per_s (HOST pointer).  `scratch8` is 8 bytes of
 * device memory whose first int is read (any value) and which is otherwise left alone.  Introspection for benchmarks;
 * the paper has no counterpart.
 */
int sr_probe_rate(int kind, void* scratch8, double* lane_ops_per_s, void* stream);

/*
 * Cycle budget of every device-side wait (mbarrier waits for copies, tensor-core results and tile hand-overs) in
 * the launches that follow, process-wide; the default is 2^31 SM cycles, about a second.  A wait that runs out
 * makes its thread block stop, wait briefly for its copies and tensor-core operations in flight, free its tensor
 * memory and return; sr_device_status then reports SR_ERR_TIMEOUT and the call's output is undefined.  Returns the
 * previous budget; cycles < 1 changes nothing.  Failure handling of this library; the paper has no counterpart.
 */
int64_t sr_set_wait_limit(int64_t cycles);

/*
 * Test hook for the failure path, host-side injection: each of the next `launches` launches of the tensor-core
 * regression kernel leaves out one barrier arrival in its first thread block, so that one of its waits runs out
 * (set a small budget with sr_set_wait_limit first).  Nothing faults or spins without bound: the block gives up
 * as described above.  0 disarms.  Returns SR_OK, or SR_ERR_SHAPE for a negative count.  The paper has no counterpart.
 */
int sr_test_lose_arrival(int launches);

/*
 * Test hook: regression calls that follow are run by kernel `kernel` (the numbering of sr_tune_result.kernel)
 * whenever that kernel supports the call, instead of the one the host rules or the tuning table pick; -1 restores
 * the rules.  Lets a test compare two kernels that serve the same call.  Returns SR_OK, or SR_ERR_SHAPE for a number
 * that names no kernel.  The paper has no counterpart.
 */
int sr_test_force_kernel(int kernel);

/*
 * Number of kernels this library has launched in this process so far (all devices, all streams).
 * Introspection for benchmarks and tests; the paper has no counterpart.
 */
int64_t sr_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SR_H_ */
