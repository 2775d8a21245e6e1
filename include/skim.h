/*
 * skim.h -- C ABI of the B200 (sm_100a) implementation of SKIM's row-clustering path
 * (SKIM: Scaled K-means clustering wIth Mixed precision, arXiv 2412.04180).
 *
 * The calls follow the paper's problem statement (Algorithm 3: inputs W, squared gradients G,
 * the bit budget and the available widths b_min..b_max; outputs labels L, centroids c, scaling
 * vector alpha):
 *
 *   skim_cluster_rows     error pre-recording: weighted 1-D K-means of every row at every
 *                         candidate width                      (Algorithm 3, first loop nest)
 *   skim_allocate_bits    greedy mixed-precision allocation     (Section 4.2, Algorithm 1)
 *   skim_quantize         labels at the allocated width, packed by width group, and the
 *                         per-row codebook                      (Algorithm 3, second loop;
 *                                                                Section 4.2, last paragraph)
 *   skim_dequantize       the fp16 matrix back from packed codes, codebooks and alpha
 *   skim_matvec           y = Wq x from the packed form   (Section 4.2, last paragraph; 4.3)
 *   skim_apply_scale      installs the scaling vector alpha: all later calls cluster
 *                         W * alpha^-1                          (Section 4.3, Algorithm 2)
 *   skim_cluster_rows_at  re-clustering at the already allocated widths inside the
 *                         grouping/scaling alternation          (Algorithm 2, outer loop)
 *   skim_scale_update     Adam steps on alpha with the labels fixed
 *                                                               (Algorithm 2, inner repeat)
 *   skim_cluster_rows_exact  the optimum of the clustering objective per row (yardstick for the iterations)
 *   skim_scale_update_lfull  the same Adam steps on the L-full loss      (Section 4.3; Section 3.4)
 *   skim_residual, skim_err_lfull   the error of a row in the L-full form, (w - wq) X X^T (w - wq)^T
 *                                                               (Section 3.4; Section 4.2; Algorithm 3)
 *
 * Conventions
 *   - Every array argument is a DEVICE pointer owned by the caller unless its comment says
 *     "host".  The library allocates no device memory: scratch comes from the workspace the
 *     caller sizes with skim_workspace_bytes and hands over with skim_set_workspace.
 *   - Work is enqueued on the stream given to skim_create and is asynchronous with respect to
 *     the host; outputs are valid once that stream has reached the end of the call's work.
 *   - Every call returns SKIM_OK (0) or a negative SKIM_ERR_* code.  Argument errors are found
 *     on the host before anything is launched.  Bad data (NaN/Inf weights, negative or NaN
 *     importance, zero or non-finite scale entries) never faults: it sets bits in a device
 *     status word that skim_get_status reads back; outputs of affected rows are unspecified.
 *   - W holds IEEE binary16 bit patterns, row-major, `ld` elements between rows (ld >= cols);
 *     importance holds binary32 with the same layout.  Rows are output channels.
 *   - bit_set (host) lists the candidate widths: strictly ascending, consecutive integers,
 *     all inside [1, SKIM_MAX_BIT].  Width b has 2^b centroids.  "sumk" below is the sum of
 *     2^b over bit_set; a row's centroid record is the concatenation of its width blocks in
 *     bit_set order, each block ascending.
 *   - The value that is clustered is x = float(W_ij) when no scale is installed, else the
 *     binary32 product float(W_ij) * r_j with r_j = 1.0f / s_j.
 */
#ifndef SKIM_H_
#define SKIM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SKIM_OK 0
#define SKIM_ERR_NULL (-1)        /* a required pointer is NULL */
#define SKIM_ERR_SHAPE (-2)       /* rows/cols/ld/iters out of range (cols above skim_max_cols included) */
#define SKIM_ERR_BITSET (-3)      /* bit_set not ascending-consecutive inside [1, SKIM_MAX_BIT] */
#define SKIM_ERR_BUDGET (-4)      /* budget outside [b_min, b_max] */
#define SKIM_ERR_WORKSPACE (-5)   /* workspace missing, too small or misaligned */
#define SKIM_ERR_CUDA (-6)        /* a CUDA runtime call failed */
#define SKIM_ERR_BAD_DATA (-7)    /* reported by skim_get_status: the status word is non-zero */
#define SKIM_ERR_SCALE (-8)       /* installed scale vector length differs from cols */
#define SKIM_ERR_ALIGN (-9)       /* an output pointer is not aligned as documented */
#define SKIM_ERR_STATIC_LIMIT (-10) /* skim_quantize_static: rows above SKIM_STATIC_MAX_ROWS */

#define SKIM_MAX_BIT 4            /* the paper caps the width at 4 bits (Section 5.1) */

/* status bits */
#define SKIM_STATUS_BAD_WEIGHT 1ull      /* NaN or Inf in W */
#define SKIM_STATUS_BAD_IMPORTANCE 2ull  /* NaN, Inf or negative importance */
#define SKIM_STATUS_BAD_SCALE 4ull       /* zero, negative or non-finite scale entry */
#define SKIM_STATUS_BAD_BITS 8ull        /* an allocated width that is not in bit_set (row skipped) */
#define SKIM_STATUS_TIMEOUT 16ull        /* an asynchronous copy did not complete within its wait limit (row skipped) */
#define SKIM_STATUS_BOUNDS 32ull         /* checked build only (-DSKIM_CHECK_BOUNDS): a computed index was out of range (access skipped) */

typedef struct skim_ctx skim_ctx;

/* Creates a context bound to `device` and to `cuda_stream` (a cudaStream_t cast to void*; NULL is
 * the legacy default stream).  The context owns only host memory.  `out` receives it. */
int skim_create(skim_ctx **out, int device, void *cuda_stream);
int skim_destroy(skim_ctx *ctx);

/* Largest `cols` the device's shared memory lets one row occupy (22 528 on B200). */
int skim_max_cols(const skim_ctx *ctx, int64_t *out);

/* Bytes of device scratch needed for matrices of up to rows x cols; `out` is a host pointer.
 * The workspace must be 256-byte aligned and stays owned by the caller.  It also stores the
 * installed scale vector, so it must outlive every call that follows skim_apply_scale.  Most of
 * it is the clustering's scratch: about 13 bytes per element for min(rows, 8192) rows (the sorted
 * rows with their prefix sums, which the sort kernel hands to the Lloyd kernel); the scale update
 * adds 8 bytes x 296 x cols of partial gradients and 520 bytes per row.
 * skim_set_workspace UNINSTALLS a scale vector that is installed (its reciprocal lives in the old
 * workspace): call skim_apply_scale again afterwards.  The caller must not release the old workspace
 * before the work already enqueued on the context's stream has finished. */
int skim_workspace_bytes(int64_t rows, int64_t cols, size_t *out);
int skim_set_workspace(skim_ctx *ctx, void *workspace, size_t bytes);

/* Section 4.3: installs the scaling vector s = alpha (device, [cols], every entry finite and
 * > 0), stored as r = 1.0f/s in the workspace; s == NULL removes it (alpha = 1).  The caller's
 * buffer is not referenced after the call's work has run. */
int skim_apply_scale(skim_ctx *ctx, const float *s, int64_t cols);

/*
 * Algorithm 3, error pre-recording.  For every row i and every width b in bit_set: weighted
 * K-means (objective sum_j g_ij (x_ij - c)^2, Section 3.2 diagonal form) with 2^b centroids,
 * index-quantile init, exactly `iters` assign/update pairs, one final assignment.
 *   centroids  out [rows][sumk] binary32; may be NULL
 *   codes      out [n_bits][rows][cols] uint8 labels of the final assignment; may be NULL
 *   err        out [rows][n_bits] binary32: the objective at the final assignment
 * iters >= 0.  1 <= cols <= skim_max_cols.  rows >= 0 (0 is a no-op).
 */
int skim_cluster_rows(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows,
                      int64_t cols, int64_t ld, const int *bit_set, int n_bits, int iters,
                      float *centroids, uint8_t *codes, float *err);

/*
 * Algorithm 2, outer loop (and Algorithm 3, second loop): as skim_cluster_rows, but row i is
 * clustered only at its allocated width row_bits[i] (device, uint8, a member of bit_set).
 *   centroids  out [rows][sumk]: only the block of the row's width is written
 *   codes      out [rows][cols] uint8, may be NULL
 *   err        out [rows] binary32, may be NULL
 */
int skim_cluster_rows_at(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows,
                         int64_t cols, int64_t ld, const uint8_t *row_bits, const int *bit_set,
                         int n_bits, int iters, float *centroids, uint8_t *codes, float *err);

/*
 * The optimum of the clustering objective (Section 3.2, diagonal form: sum_j g_ij (x_ij - c)^2 over all
 * assignments to 2^b centroids), where skim_cluster_rows runs the Lloyd iterations of Algorithm 3, which stop
 * in a local optimum: the yardstick for them, at the same interface.  In one dimension the optimal clusters are
 * intervals of the sorted row; a dynamic programme over the split points finds them (cols * log cols cost
 * evaluations per centroid, all widths sharing the layers).
 *   centroids  out [rows][sumk] binary32: the weighted means of the optimal intervals, ascending (an interval
 *              whose importances are all zero takes the mean of its first and last value)
 *   err        out [rows][n_bits] binary32: the optimum
 * Rows with at most 2^b distinct values get those values and error 0, as in skim_cluster_rows.  Where two
 * partitions cost the same up to rounding either may be returned.  An installed scale vector applies.
 *   scratch    device, 256-byte aligned, at least skim_cluster_exact_bytes(ctx, rows, cols) bytes
 *              (about 74 bytes per column for each of min(rows, 3 x SM count) rows in flight)
 */
int skim_cluster_exact_bytes(const skim_ctx *ctx, int64_t rows, int64_t cols, size_t *out);
int skim_cluster_rows_exact(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                            int64_t ld, const int *bit_set, int n_bits, void *scratch, size_t scratch_bytes,
                            float *centroids, float *err);

/*
 * Algorithm 1.  All rows start at b_min; the row with the largest error reduction
 * err[i][b_i] - err[i][b_i+1] (differences taken in binary64; lowest row index on ties) gains a
 * bit until the total is T = floor(rows * budget + 1e-6).  Reductions may be negative.
 *   err         [rows][n_bits] binary32 (column u is width bit_set[u])
 *   bits        out [rows] uint8
 *   total_bits  host out, may be NULL: T (computed on the host, no synchronisation)
 */
int skim_allocate_bits(skim_ctx *ctx, const float *err, int64_t rows, const int *bit_set, int n_bits,
                       double budget, uint8_t *bits, int64_t *total_bits);

/*
 * Algorithm 1 with its stopping rule as printed: bits are handed out until the total reaches
 * rows * budget, so a non-integer product is rounded UP, T = ceil(rows * budget - 1e-6), and the
 * average may exceed the budget by less than 1/rows of a bit.  Otherwise as skim_allocate_bits, which
 * rounds down to keep Section 4.2's constraint (average <= budget).
 */
int skim_allocate_bits_until(skim_ctx *ctx, const float *err, int64_t rows, const int *bit_set, int n_bits,
                             double budget, uint8_t *bits, int64_t *total_bits);

/*
 * The allocation variant of the appendix on other model families (additional perplexity results):
 * the allocation starts from the budget rounded down, floor(budget), for every row instead of from
 * b_min, and Algorithm 1 hands out only the remaining T - rows * floor(budget) bits.  With an integer
 * budget nothing remains: every row gets exactly that width, i.e. mixed precision is off.
 * Arguments, tie rule, T and errors as for skim_allocate_bits.
 */
int skim_allocate_bits_floor(skim_ctx *ctx, const float *err, int64_t rows, const int *bit_set, int n_bits,
                             double budget, uint8_t *bits, int64_t *total_bits);

/*
 * The exact solution of Section 4.2's allocation problem -- minimise the summed error subject to the
 * bit budget -- by the dynamic programme the paper names as precise but quadratic: the yardstick for
 * Algorithm 1 (how much error the greedy leaves on the table), not a step of the quantisation path.
 * The total is the greedy's T = floor(rows * budget + 1e-6); ties go to the smaller width.
 * Cost: rows * (T - rows * b_min) * n_bits additions on one SM (4096 rows at 3.0 bits: a few ms).
 *   scratch     device, 256-byte aligned, at least skim_allocate_optimal_bytes (it holds one
 *               byte per row and state: rows * (T - rows*b_min + 1) bytes, plus two value rows)
 *   bits        out [rows] uint8;  total_bits  host out, may be NULL
 *   cost        device out, may be NULL: the minimum, one binary64 (the errors added in row order)
 */
int skim_allocate_optimal_bytes(int64_t rows, const int *bit_set, int n_bits, double budget, size_t *out);
int skim_allocate_optimal(skim_ctx *ctx, const float *err, int64_t rows, const int *bit_set, int n_bits,
                          double budget, void *scratch, size_t scratch_bytes, uint8_t *bits,
                          int64_t *total_bits, double *cost);

/* Packed layout (host-only helper): 32-bit words per packed row of each width,
 * ceil(cols*b/32) rounded up to a multiple of 4, and the byte size that is enough for any
 * allocation (every row at the largest width).  Outputs are host pointers; either may be NULL. */
int skim_packed_layout(int64_t rows, int64_t cols, const int *bit_set, int n_bits,
                       int64_t *row_stride_words, size_t *max_packed_bytes);

/*
 * Algorithm 3, final labels and codebooks, packed as Section 4.2 describes: rows of equal width
 * are gathered (ascending width, ascending row index inside a group) and stored back to back.
 *   bits        [rows] uint8 allocated widths
 *   centroids   [rows][sumk] binary32 (from skim_cluster_rows or skim_cluster_rows_at)
 *   packed      out, 16-byte aligned: a packed row is a little-endian bit stream, element j in
 *               bits [j*b, (j+1)*b) of the row, zero padded to the row stride
 *   row_order   out [rows] int32: source row of every packed row
 *   group_info  out [2*(n_bits+1)] int64: first packed row of every width group, then the
 *               32-bit-word offset of every group inside `packed` (last entries: totals)
 *   lut         out [rows][2^b_max] binary16 bit patterns of the row's centroids, round to
 *               nearest even, entries beyond 2^b_i repeat the last one
 * The label of an element is the number of midpoints (c_j + c_{j+1})/2 that lie strictly below it.
 */
int skim_quantize(skim_ctx *ctx, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld,
                  const uint8_t *bits, const float *centroids, const int *bit_set, int n_bits,
                  uint32_t *packed, int32_t *row_order, int64_t *group_info, uint16_t *lut);

/*
 * skim_quantize for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this call; it exists for integration reasons only.)
 *
 * Some users of this library run where cudaMalloc is off limits: inside another framework's
 * allocator or plugin callback, in a process whose device memory was planned and handed out in
 * full at start-up, or in a latency-critical loop where an allocation's implicit device
 * synchronisation is not acceptable.  They can neither create a workspace nor let a library do
 * it.  This variant needs no context and no workspace: the scratch that skim_quantize keeps in
 * the workspace (one packed-row index per row and a status word) lives in a fixed array inside
 * the library image, 256 + 4 * SKIM_STATIC_MAX_ROWS bytes on every GPU that loads the library,
 * held until the process exits.  It calls no cudaMalloc/cudaFree and no allocating routine.
 *
 *   - Same inputs, outputs, layout and labels as skim_quantize with no scale vector installed
 *     (alpha = 1); all array arguments are device pointers, bit_set is a host pointer.
 *   - Runs on the CURRENT device, on `cuda_stream` (a cudaStream_t cast to void*).
 *   - rows must not exceed SKIM_STATIC_MAX_ROWS, else SKIM_ERR_STATIC_LIMIT and nothing runs.
 *   - The first call on a device looks up the array's device address (one
 *     cudaGetSymbolAddress, cached per device); make that first call outside any stream capture.
 *     The cached address does not survive cudaDeviceReset or the destruction of the device's
 *     primary context: a process that does either must not call this function afterwards.
 *   - All calls on a device share the one array, and it keeps the previous call's contents
 *     (the call clears what it needs at zero).  Two calls that overlap on the GPU -- different
 *     streams, or different host threads -- race on it: serialise them.
 *   - A width outside bit_set is skipped, as in skim_quantize; it shows as
 *     group_info[n_bits] < rows (there is no context to read a status word from).
 */
#define SKIM_STATIC_MAX_ROWS 65536
int skim_quantize_static(void *cuda_stream, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld,
                         const uint8_t *bits, const float *centroids, const int *bit_set, int n_bits,
                         uint32_t *packed, int32_t *row_order, int64_t *group_info, uint16_t *lut);

/*
 * Unpacking (Section 4.2, last paragraph: rows of equal width are stored together and unpacked
 * group by group; Section 4 overview and Section 4.3: the dequantised weight is the codebook
 * entry of its label times the scaling vector, Wq = Quant(W * alpha^-1) * alpha).
 * Inputs are the outputs of skim_quantize: packed, row_order [rows], group_info [2*(n_bits+1)],
 * lut [rows][2^b_max] (indexed by SOURCE row), all device pointers; s (device, [cols], may be
 * NULL for alpha = 1) is the scaling vector itself, not its reciprocal.  No workspace is used.
 *   out  [rows][ld_out] binary16, source-row order:
 *        out[i][j] = binary16( float(lut[i][code_ij]) * s_j ), the product taken in binary32 and
 *        rounded to nearest even once more; with s == NULL the codebook entry itself.
 * Rows that skim_quantize skipped (width outside bit_set) are left untouched.
 * cols is limited by shared memory (the per-column vector of a block sits there: about 58 000 on
 * B200); ld_out >= cols.
 */
int skim_dequantize(skim_ctx *ctx, const uint32_t *packed, const int32_t *row_order, const int64_t *group_info,
                    const uint16_t *lut, const float *s, int64_t rows, int64_t cols, const int *bit_set,
                    int n_bits, uint16_t *out, int64_t ld_out);

/*
 * y = Wq x straight from the packed form, Wq as defined for skim_dequantize but never rounded to
 * binary16 or stored: y_i = sum_j float(lut[i][code_ij]) * z_j with z_j = float(x_j) * s_j in
 * binary32 (z = x when s == NULL).  The sum is accumulated in binary32 (per lane in element
 * order, then a 5-level tree), so |y_i - exact| <= (cols/32 + 8) * 2^-24 * sum_j |term_ij|.
 *   x  [cols] binary16 bit patterns (device);  y  out [rows] binary32, source-row order (device)
 */
int skim_matvec(skim_ctx *ctx, const uint32_t *packed, const int32_t *row_order, const int64_t *group_info,
                const uint16_t *lut, const float *s, const uint16_t *x, int64_t rows, int64_t cols,
                const int *bit_set, int n_bits, float *y);

/*
 * Algorithm 2, inner repeat: `steps` Adam updates (Section 5.1: learning rate lr0, multiplied
 * by `decay` every `decay_every` steps; betas 0.9/0.999, eps 1e-8) of the scaling vector with the
 * labels fixed, on loss = sum g_ij (W_ij - alpha_j c_{i,l_ij})^2 with importance-weighted
 * centroids c of W * alpha^-1 re-fitted at every step.
 *   labels      [rows][cols] uint8 (as written by skim_cluster_rows_at)
 *   alpha       in/out [cols] binary32, every entry > 0
 *   loss_trace  out, may be NULL: [steps] binary64, the loss at the alpha each step started from
 * Does not install alpha; call skim_apply_scale(alpha) afterwards to cluster with it.
 */
int skim_scale_update(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows,
                      int64_t cols, int64_t ld, const uint8_t *labels, float *alpha, int steps,
                      float lr0, float decay, int decay_every, double *loss_trace);

/*
 * L-full error (Section 3.4: the layer-wise objective of row i is (w_i - wq_i) X X^T (w_i - wq_i)^T, named
 * L-full; Section 4.2 and Algorithm 3 use it for the error table; Section 4.3: wq = replace(c, l) * alpha).
 * Two calls: the residual, then the quadratic form with H = X X^T.
 *
 * skim_residual:  D[i][j] = binary16( (float(W_ij) - c_{i,l_ij} * alpha_j) * 2^exp2 )
 *   label l_ij by the packer's rule (number of midpoints strictly below the clustered value) among the
 *   centroids of the row's width block; the product c * alpha and the difference are taken in binary32, the
 *   scaling by 2^exp2 is exact, one rounding to nearest even to binary16 (overflow gives infinity: pick exp2
 *   so that |residual| * 2^exp2 < 65504; 8 suits weights of magnitude below 1).
 *   centroids  [rows][sumk] binary32;  row_bits [rows] uint8 or NULL (then every row uses `width`)
 *   s          the scaling vector alpha itself (device, [cols]) or NULL.  With s != NULL the same vector must be
 *              installed (skim_apply_scale), else SKIM_ERR_SCALE: the labels need its reciprocal.
 *   D          out [rows][ldd] binary16, ldd >= cols; for skim_err_lfull: 16-byte aligned, ldd % 8 == 0
 *   0 <= exp2 <= 24.  A width outside bit_set sets SKIM_STATUS_BAD_BITS and leaves the row untouched.
 *
 * skim_err_lfull:  err[i * err_stride] = ( sum_j sum_k D_ij H_jk D_ik ) / 4^exp2
 *   H          [cols][ldh] binary16 (device), the Gram matrix X X^T of the layer's inputs; only its symmetric
 *              part matters.  16-byte aligned, ldh % 8 == 0.  cols % 8 == 0.
 *   scratch    device, 256-byte aligned, at least skim_err_lfull_bytes(rows, cols) bytes
 *   err        out binary32; err_stride elements between rows (n_bits to fill one column of the error table)
 * The products are exact in binary32 and are accumulated in binary32 by the tensor cores (cols terms per output
 * of D H, then cols terms per row), the sums per tile (per range of K where a tile of the last, partly filled round
 * of tiles is cut along K) in binary64:  |err - exact| <= (2 cols + 600) * 2^-24 *
 * sum_jk |D_ij H_jk D_ik| / 4^exp2.  Needs the workspace (status word).
 */
int skim_residual(skim_ctx *ctx, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld, const float *centroids,
                  const uint8_t *row_bits, int width, const int *bit_set, int n_bits, const float *s, int exp2,
                  uint16_t *D, int64_t ldd);
int skim_err_lfull_bytes(int64_t rows, int64_t cols, size_t *out);
int skim_err_lfull(skim_ctx *ctx, const uint16_t *D, int64_t rows, int64_t cols, int64_t ldd, const uint16_t *H,
                   int64_t ldh, int exp2, void *scratch, size_t scratch_bytes, float *err, int64_t err_stride);

/*
 * skim_scale_update on the L-full loss (Section 4.3: "the loss calculation adopts the L-full form"; the form itself
 * in Section 3.4):  loss = sum_i d_i H d_i^T,  d_ij = W_ij - alpha_j c_{i,l_ij},  with the importance-weighted centroids
 * c of W * alpha^-1 re-fitted at every step as in skim_scale_update, and H = X X^T as for skim_err_lfull.  Per step the
 * residual goes through the tensor-core contraction as binary16(float(d) * 2^exp2) (the gradient treats that
 * rounding as the identity), Y = D H is kept in binary32, everything else is binary64.
 *   labels, alpha, steps, lr0, decay, decay_every, loss_trace: as for skim_scale_update
 *   H        [cols][ldh] binary16 (device), 16-byte aligned, ldh % 8 == 0
 *   scratch  device, 256-byte aligned, at least skim_scale_lfull_bytes(rows, cols) bytes (6 bytes per element
 *            for the residual and the product, plus the contraction's partial sums)
 * cols % 8 == 0, ld % 8 == 0, W, importance and labels 16-byte aligned (SKIM_ERR_ALIGN otherwise).
 */
int skim_scale_lfull_bytes(int64_t rows, int64_t cols, size_t *out);
int skim_scale_update_lfull(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                            int64_t ld, const uint8_t *labels, const uint16_t *H, int64_t ldh, float *alpha, int steps,
                            float lr0, float decay, int decay_every, int exp2, void *scratch, size_t scratch_bytes,
                            double *loss_trace);

/*
 * The whole path from HOST buffers: copies W and importance to the device staging area, runs
 * skim_cluster_rows, skim_allocate_bits and skim_quantize, and copies the results back, then
 * waits for the stream.  `staging` is device memory of at least skim_host_staging_bytes bytes,
 * 256-byte aligned.  Host outputs (any may be NULL): err [rows][n_bits], bits [rows], packed
 * (skim_packed_layout max bytes), row_order [rows], group_info [2*(n_bits+1)],
 * lut [rows][2^b_max].
 */
int skim_host_staging_bytes(int64_t rows, int64_t cols, const int *bit_set, int n_bits, size_t *out);
int skim_quantize_matrix_host(skim_ctx *ctx, const uint16_t *W_host, const float *importance_host,
                              int64_t rows, int64_t cols, const int *bit_set, int n_bits, int iters,
                              double budget, void *staging, size_t staging_bytes, float *err_host,
                              uint8_t *bits_host, uint32_t *packed_host, int32_t *row_order_host,
                              int64_t *group_info_host, uint16_t *lut_host);

/* Reads and clears the device status word (synchronises the stream).  Returns SKIM_OK when it
 * was zero, SKIM_ERR_BAD_DATA otherwise; `flags` (host, may be NULL) receives the bits. */
int skim_get_status(skim_ctx *ctx, uint64_t *flags);

/* Number of kernel launches the context has issued so far (host counter). */
int64_t skim_launch_count(const skim_ctx *ctx);

/*
 * Measurement aid (no counterpart in the paper).  skim_cluster_rows and skim_cluster_rows_at run,
 * per chunk of rows, a row-sorting kernel followed by a Lloyd kernel (Algorithm 3, first loop
 * nest).  With timing enabled the context records a CUDA event on its stream before, between and
 * after the two, for up to 256 chunks; further chunks go untimed.  skim_kernel_timing(ctx, 1)
 * starts a fresh series (the events are created on the first call; no device memory is involved),
 * skim_kernel_timing(ctx, 0) stops recording.  skim_kernel_times waits for the last recorded
 * event and returns the summed durations in milliseconds and the number of chunks they cover
 * (host pointers, any may be NULL).
 */
int skim_kernel_timing(skim_ctx *ctx, int enable);
int skim_kernel_times(skim_ctx *ctx, double *sort_ms, double *lloyd_ms, int64_t *chunks);

/*
 * Measurement aids for the iteration count (no counterpart in the paper, which states no stopping
 * rule).  The clustering runs exactly `iters` assign/update pairs per row, except that a row stops as
 * soon as an assignment moved no boundary: every later pair would reproduce the same state bit for
 * bit, so the result is the same.  skim_early_exit(ctx, 0) switches that shortcut off (all rows run
 * all `iters` pairs; same output, more time), skim_early_exit(ctx, 1) restores the default.
 * While skim_kernel_timing is enabled the Lloyd kernel also adds up the pairs each row really ran;
 * skim_lloyd_iterations reads and clears that count (it waits for the stream): `iterations` = pairs
 * summed over rows, `rows` = rows counted (host pointers, either may be NULL).
 */
int skim_early_exit(skim_ctx *ctx, int enable);
int skim_lloyd_iterations(skim_ctx *ctx, int64_t *iterations, int64_t *rows);

const char *skim_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* SKIM_H_ */
