// Internal declarations shared by the translation units of libskim.so.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "skim.h"

#define SKIM_MAX_NBITS SKIM_MAX_BIT
#define SKIM_HOST_CHUNKS 8   // row chunks of the host-buffer entry point
#define SKIM_MAX_SUMK 30  // 2 + 4 + 8 + 16: one warp lane per centroid
#define SKIM_TIMING_SLOTS 256   // clustering chunks whose kernel times skim_kernel_timing can hold

struct skim_ctx {
    int device;
    cudaStream_t stream;
    int sm_count;
    int max_smem_optin;   // bytes of dynamic shared memory one block may opt into
    void *ws;             // caller's workspace
    size_t ws_bytes;
    bool scaled;          // a scale vector is installed
    int64_t scale_cols;
    int64_t launches;
    // host-buffer entry point: a second stream for the host-to-device copies, so that the copy
    // of one row chunk runs under the clustering of the previous one (created on first use)
    cudaStream_t copy_stream;
    cudaEvent_t copy_done[SKIM_HOST_CHUNKS];
    cudaEvent_t main_idle;
    bool copy_ready;
    // optional kernel timing: events before the sort kernel, between the two kernels and after
    // the Lloyd kernel of every clustering chunk, on the context's stream
    bool early_exit;      // rows stop iterating once no boundary moved (default)
    bool timing;
    bool timing_ready;
    int timing_used;
    cudaEvent_t timing_ev[SKIM_TIMING_SLOTS][3];
};

// Workspace layout (all offsets 256-byte aligned), carved per call for the call's (rows, cols).
// The status word and the reciprocal scale sit at fixed offsets, so they persist across calls.
struct SkimWorkspace {
    unsigned long long *status;  // word 0: status bits; words 1, 2: Lloyd iterations run and rows counted (skim_lloyd_iterations)
    float *rscale;               // [cols]     reciprocal of the installed scale vector
    int32_t *row_pos;            // [rows]     packed-row index of every source row
    double *alpha64;             // [cols]     scale-update master copy of alpha
    double *alpha_il;            // [cols rounded up to 256]  the same values in the order the row-wise kernels load them
    double *adam_m;              // [cols]
    double *adam_v;              // [cols]
    double *loss_part;           // [rows]     scale update: loss of every row
    double *grad_part;           // [SKIM_SCALE_MAX_CTAS][cols]  partial gradients of the row ranges
    double *scale_const;         // [rows][16][2]  scale update: per-cluster constants (sum g, sum g w^2)
    double *scale_cq;            // [rows][16][2]  scale update: per-cluster centroid and gradient factor
    unsigned char *cluster_scratch;  // [min(rows, SKIM_CLUSTER_CHUNK_ROWS)] row records of the clustering
    size_t bytes;
};

#define SKIM_SCALE_MAX_CTAS 296
#define SKIM_CLUSTER_CHUNK_ROWS 8192   // rows clustered per sort-kernel / Lloyd-kernel pair

// Upper bound of one row record of the clustering: 128-byte header, 96 bytes per group of 8
// elements, group index 0.5 B per element, segment table, plus rounding.
__host__ __device__ static inline size_t skim_cluster_record_bytes(int64_t cols)
{
    const size_t m8 = ((size_t)cols + 7) & ~(size_t)7;
    return (13 * m8 + 1024 + 127) & ~(size_t)127;
}

static inline size_t skim_align256(size_t v) { return (v + 255) & ~(size_t)255; }

static inline SkimWorkspace skim_carve(void *base, int64_t rows, int64_t cols)
{
    SkimWorkspace w;
    char *p = (char *)base;
    size_t off = 0;
    auto take = [&](size_t bytes) { char *q = p ? p + off : nullptr; off += skim_align256(bytes); return q; };
    w.status = (unsigned long long *)take(256);
    w.rscale = (float *)take((size_t)cols * 4);
    w.row_pos = (int32_t *)take((size_t)rows * 4);
    w.alpha64 = (double *)take((size_t)cols * 8);
    w.alpha_il = (double *)take((((size_t)cols + 255) & ~(size_t)255) * 8);
    w.adam_m = (double *)take((size_t)cols * 8);
    w.adam_v = (double *)take((size_t)cols * 8);
    w.loss_part = (double *)take((size_t)(rows > SKIM_SCALE_MAX_CTAS ? rows : SKIM_SCALE_MAX_CTAS) * 8);
    w.grad_part = (double *)take((size_t)SKIM_SCALE_MAX_CTAS * (size_t)cols * 8);
    w.scale_const = (double *)take((size_t)rows * 16 * 2 * 8);
    w.scale_cq = (double *)take((size_t)rows * 16 * 2 * 8);
    w.cluster_scratch = (unsigned char *)take((size_t)(rows < SKIM_CLUSTER_CHUNK_ROWS ? rows : SKIM_CLUSTER_CHUNK_ROWS) *
                                              skim_cluster_record_bytes(cols));
    w.bytes = off;
    return w;
}

// Index checks of the checked build (nvcc -DSKIM_CHECK_BOUNDS; build.py builds it as libskim_checked.so).
// Every index into shared memory, a row record or a scratch list that is COMPUTED from data (a scatter
// position, a counter slot, a searched group, a gathered column) goes through SKIM_IDX: in the checked
// build an index outside [0, n) sets SKIM_STATUS_BOUNDS in the status word and the access is skipped
// (never a trap); in the normal build the macro is the constant true and costs nothing.
#ifdef SKIM_CHECK_BOUNDS
__device__ __forceinline__ bool skim_index_ok(long long i, long long n, unsigned long long *status)
{
    if (i >= 0 && i < n) return true;
    if (status) atomicOr(status, (unsigned long long)SKIM_STATUS_BOUNDS);
    return false;
}
#define SKIM_IDX(i, n, status) skim_index_ok((long long)(i), (long long)(n), (status))
#else
#define SKIM_IDX(i, n, status) true
#endif

// Validated description of a bit set.
struct SkimBits {
    int n_bits;
    int b_min;
    int b_max;
    int sumk;
};

int skim_check_bits(const int *bit_set, int n_bits, SkimBits *out);

#define SKIM_CUDA_OK(expr)                         \
    do {                                           \
        cudaError_t e_ = (expr);                   \
        if (e_ != cudaSuccess) return SKIM_ERR_CUDA; \
    } while (0)

// Launchers implemented in the kernel translation units.  All return SKIM_OK or SKIM_ERR_*.
// exact_scratch == nullptr: Lloyd iterations (Algorithm 3); else the exact optimum of every row (skim_exact.cu)
int skim_launch_cluster(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows,
                        int64_t cols, int64_t ld, const uint8_t *row_bits, const SkimBits &bits,
                        int iters, float *centroids, uint8_t *codes, float *err, void *exact_scratch = nullptr);
size_t skim_exact_slot_bytes(int64_t cols);
int skim_exact_slots(const skim_ctx *ctx, int64_t rows);
int skim_cluster_max_cols(int max_smem_optin, int64_t *out);
int skim_launch_reciprocal(skim_ctx *ctx, const float *s, int64_t cols);
int skim_launch_allocate(skim_ctx *ctx, const float *err, int64_t rows, const SkimBits &bits, int first_col,
                         int64_t K, uint8_t *out_bits);
size_t skim_allocate_optimal_scratch(int64_t rows, int64_t K);
int skim_launch_allocate_optimal(skim_ctx *ctx, const float *err, int64_t rows, const SkimBits &bits, int64_t K,
                                 void *scratch, uint8_t *out_bits, double *cost);
int skim_launch_quantize(skim_ctx *ctx, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld,
                         const uint8_t *bits, const float *centroids, const SkimBits &bs,
                         uint32_t *packed, int32_t *row_order, int64_t *group_info, uint16_t *lut);
int skim_launch_dequantize(skim_ctx *ctx, const uint32_t *packed, const int32_t *row_order, const int64_t *group_info,
                           const uint16_t *lut, const float *s, int64_t rows, int64_t cols, const SkimBits &bs,
                           uint16_t *out, int64_t ld_out);
int skim_launch_matvec(skim_ctx *ctx, const uint32_t *packed, const int32_t *row_order, const int64_t *group_info,
                       const uint16_t *lut, const float *s, const uint16_t *x, int64_t rows, int64_t cols,
                       const SkimBits &bs, float *y);
int skim_launch_scale_update(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows,
                             int64_t cols, int64_t ld, const uint8_t *labels, float *alpha, int steps,
                             float lr0, float decay, int decay_every, double *loss_trace);

int skim_launch_residual(skim_ctx *ctx, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld, const float *centroids,
                         const uint8_t *row_bits, int width, const SkimBits &bs, const float *s, int exp2, uint16_t *D,
                         int64_t ldd);
size_t skim_lfull_scratch_bytes(int64_t rows, int64_t cols);
// Y (optional): the product D H itself, [rows][ldy] binary32; err64 (optional): the row errors in binary64
int skim_launch_err_lfull(skim_ctx *ctx, const uint16_t *D, int64_t rows, int64_t cols, int64_t ldd, const uint16_t *H,
                          int64_t ldh, int exp2, void *scratch, float *err, int64_t err_stride, float *Y = nullptr,
                          int64_t ldy = 0, double *err64 = nullptr);
size_t skim_scale_lfull_scratch_bytes(int64_t rows, int64_t cols);
int skim_launch_scale_update_lfull(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                                   int64_t ld, const uint8_t *labels, const uint16_t *H, int64_t ldh, float *alpha,
                                   int steps, float lr0, float decay, int decay_every, int exp2, void *scratch,
                                   double *loss_trace);

__host__ __device__ static inline int64_t skim_row_stride_words(int64_t cols, int b)
{
    int64_t w = (cols * (int64_t)b + 31) / 32;
    return (w + 3) / 4 * 4;
}
