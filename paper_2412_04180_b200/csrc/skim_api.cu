// Host side of the C ABI: context, argument validation, workspace bookkeeping, dispatch.
#include <math.h>
#include <new>

#include "skim_internal.cuh"

int skim_check_bits(const int *bit_set, int n_bits, SkimBits *out)
{
    if (!bit_set) return SKIM_ERR_NULL;
    if (n_bits < 1 || n_bits > SKIM_MAX_NBITS) return SKIM_ERR_BITSET;
    int sumk = 0;
    for (int b = 0; b < n_bits; ++b) {
        if (bit_set[b] < 1 || bit_set[b] > SKIM_MAX_BIT) return SKIM_ERR_BITSET;
        if (b && bit_set[b] != bit_set[b - 1] + 1) return SKIM_ERR_BITSET;
        sumk += 1 << bit_set[b];
    }
    out->n_bits = n_bits;
    out->b_min = bit_set[0];
    out->b_max = bit_set[n_bits - 1];
    out->sumk = sumk;
    return SKIM_OK;
}

namespace {

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

int check_matrix(const skim_ctx *ctx, int64_t rows, int64_t cols, int64_t ld)
{
    if (rows < 0 || rows > 0x7fffffff || cols < 1 || ld < cols) return SKIM_ERR_SHAPE;
    int64_t maxc = 0;
    skim_cluster_max_cols(ctx->max_smem_optin, &maxc);
    if (cols > maxc) return SKIM_ERR_SHAPE;
    return SKIM_OK;
}

int check_workspace(const skim_ctx *ctx, int64_t rows, int64_t cols)
{
    if (!ctx->ws) return SKIM_ERR_WORKSPACE;
    const SkimWorkspace need = skim_carve(nullptr, rows, cols);
    return need.bytes <= ctx->ws_bytes ? SKIM_OK : SKIM_ERR_WORKSPACE;
}

}  // namespace

extern "C" {

int skim_create(skim_ctx **out, int device, void *cuda_stream)
{
    if (!out) return SKIM_ERR_NULL;
    *out = nullptr;
    int count = 0;
    SKIM_CUDA_OK(cudaGetDeviceCount(&count));
    if (device < 0 || device >= count) return SKIM_ERR_SHAPE;
    skim_ctx *ctx = new (std::nothrow) skim_ctx();
    if (!ctx) return SKIM_ERR_CUDA;
    ctx->device = device;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->ws = nullptr;
    ctx->ws_bytes = 0;
    ctx->scaled = false;
    ctx->scale_cols = 0;
    ctx->launches = 0;
    ctx->copy_ready = false;
    ctx->early_exit = true;
    ctx->timing = false;
    ctx->timing_ready = false;
    ctx->timing_used = 0;
    if (cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&ctx->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess) {
        delete ctx;
        return SKIM_ERR_CUDA;
    }
    *out = ctx;
    return SKIM_OK;
}

int skim_destroy(skim_ctx *ctx)
{
    if (ctx && ctx->copy_ready) {
        DeviceGuard guard(ctx->device);
        cudaStreamDestroy(ctx->copy_stream);
        for (int k = 0; k < SKIM_HOST_CHUNKS; ++k) cudaEventDestroy(ctx->copy_done[k]);
        cudaEventDestroy(ctx->main_idle);
    }
    if (ctx && ctx->timing_ready) {
        DeviceGuard guard(ctx->device);
        for (int k = 0; k < SKIM_TIMING_SLOTS; ++k)
            for (int e = 0; e < 3; ++e) cudaEventDestroy(ctx->timing_ev[k][e]);
    }
    delete ctx;
    return SKIM_OK;
}

int skim_max_cols(const skim_ctx *ctx, int64_t *out)
{
    if (!ctx || !out) return SKIM_ERR_NULL;
    return skim_cluster_max_cols(ctx->max_smem_optin, out);
}

int skim_workspace_bytes(int64_t rows, int64_t cols, size_t *out)
{
    if (!out) return SKIM_ERR_NULL;
    if (rows < 0 || cols < 1) return SKIM_ERR_SHAPE;
    *out = skim_carve(nullptr, rows, cols).bytes;
    return SKIM_OK;
}

int skim_set_workspace(skim_ctx *ctx, void *workspace, size_t bytes)
{
    if (!ctx || !workspace) return SKIM_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || bytes < 512) return SKIM_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    ctx->ws = workspace;
    ctx->ws_bytes = bytes;
    ctx->scaled = false;
    ctx->scale_cols = 0;
    SKIM_CUDA_OK(cudaMemsetAsync(workspace, 0, 256, ctx->stream));   // status word
    return SKIM_OK;
}

int skim_apply_scale(skim_ctx *ctx, const float *s, int64_t cols)
{
    if (!ctx) return SKIM_ERR_NULL;
    if (!s) {
        ctx->scaled = false;
        ctx->scale_cols = 0;
        return SKIM_OK;
    }
    if (cols < 1) return SKIM_ERR_SHAPE;
    int rc = check_workspace(ctx, 0, cols);
    if (rc) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    rc = skim_launch_reciprocal(ctx, s, cols);
    if (rc) return rc;
    ctx->scaled = true;
    ctx->scale_cols = cols;
    return SKIM_OK;
}

static int cluster_common(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                          int64_t ld, const uint8_t *row_bits, const int *bit_set, int n_bits, int iters,
                          float *centroids, uint8_t *codes, float *err)
{
    if (!ctx || !W || !importance) return SKIM_ERR_NULL;
    SkimBits bits;
    int rc = skim_check_bits(bit_set, n_bits, &bits);
    if (rc) return rc;
    rc = check_matrix(ctx, rows, cols, ld);
    if (rc) return rc;
    if (iters < 0) return SKIM_ERR_SHAPE;
    rc = check_workspace(ctx, rows, cols);
    if (rc) return rc;
    if (ctx->scaled && ctx->scale_cols != cols) return SKIM_ERR_SCALE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_cluster(ctx, W, importance, rows, cols, ld, row_bits, bits, iters, centroids, codes, err);
}

int skim_cluster_rows(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                      int64_t ld, const int *bit_set, int n_bits, int iters, float *centroids, uint8_t *codes,
                      float *err)
{
    if (!err) return SKIM_ERR_NULL;
    return cluster_common(ctx, W, importance, rows, cols, ld, nullptr, bit_set, n_bits, iters, centroids, codes, err);
}

int skim_cluster_rows_at(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                         int64_t ld, const uint8_t *row_bits, const int *bit_set, int n_bits, int iters,
                         float *centroids, uint8_t *codes, float *err)
{
    if (!row_bits || !centroids) return SKIM_ERR_NULL;
    return cluster_common(ctx, W, importance, rows, cols, ld, row_bits, bit_set, n_bits, iters, centroids, codes, err);
}

int skim_cluster_exact_bytes(const skim_ctx *ctx, int64_t rows, int64_t cols, size_t *out)
{
    if (!ctx || !out) return SKIM_ERR_NULL;
    int rc = check_matrix(ctx, rows, cols, cols);
    if (rc) return rc;
    *out = skim_align256((size_t)skim_exact_slots(ctx, rows > 0 ? rows : 1) * skim_exact_slot_bytes(cols));
    return SKIM_OK;
}

int skim_cluster_rows_exact(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                            int64_t ld, const int *bit_set, int n_bits, void *scratch, size_t scratch_bytes,
                            float *centroids, float *err)
{
    if (!ctx || !W || !importance || !scratch || !centroids || !err) return SKIM_ERR_NULL;
    SkimBits bits;
    int rc = skim_check_bits(bit_set, n_bits, &bits);
    if (rc) return rc;
    rc = check_matrix(ctx, rows, cols, ld);
    if (rc) return rc;
    rc = check_workspace(ctx, rows, cols);
    if (rc) return rc;
    if (ctx->scaled && ctx->scale_cols != cols) return SKIM_ERR_SCALE;
    if ((reinterpret_cast<uintptr_t>(scratch) & 255u) != 0 ||
        scratch_bytes < (size_t)skim_exact_slots(ctx, rows > 0 ? rows : 1) * skim_exact_slot_bytes(cols))
        return SKIM_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_cluster(ctx, W, importance, rows, cols, ld, nullptr, bits, 0, centroids, nullptr, err, scratch);
}

int skim_allocate_bits(skim_ctx *ctx, const float *err, int64_t rows, const int *bit_set, int n_bits, double budget,
                       uint8_t *bits_out, int64_t *total_bits)
{
    if (!ctx || !err || !bits_out) return SKIM_ERR_NULL;
    SkimBits bits;
    int rc = skim_check_bits(bit_set, n_bits, &bits);
    if (rc) return rc;
    if (rows < 1 || rows > 0x7fffffff) return SKIM_ERR_SHAPE;
    if (!(budget >= (double)bits.b_min && budget <= (double)bits.b_max)) return SKIM_ERR_BUDGET;
    const int64_t T = (int64_t)floor((double)rows * budget + 1e-6);
    const int64_t K = T - rows * (int64_t)bits.b_min;
    if (K < 0 || K > rows * (int64_t)(bits.b_max - bits.b_min)) return SKIM_ERR_BUDGET;
    if (total_bits) *total_bits = T;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_allocate(ctx, err, rows, bits, 0, K, bits_out);
}

int skim_allocate_bits_until(skim_ctx *ctx, const float *err, int64_t rows, const int *bit_set, int n_bits,
                             double budget, uint8_t *bits_out, int64_t *total_bits)
{
    if (!ctx || !err || !bits_out) return SKIM_ERR_NULL;
    SkimBits bits;
    int rc = skim_check_bits(bit_set, n_bits, &bits);
    if (rc) return rc;
    if (rows < 1 || rows > 0x7fffffff) return SKIM_ERR_SHAPE;
    if (!(budget >= (double)bits.b_min && budget <= (double)bits.b_max)) return SKIM_ERR_BUDGET;
    int64_t T = (int64_t)ceil((double)rows * budget - 1e-6);      // the first total that is >= rows * budget
    if (T < rows * (int64_t)bits.b_min) T = rows * (int64_t)bits.b_min;
    if (T > rows * (int64_t)bits.b_max) T = rows * (int64_t)bits.b_max;
    if (total_bits) *total_bits = T;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_allocate(ctx, err, rows, bits, 0, T - rows * (int64_t)bits.b_min, bits_out);
}

int skim_allocate_bits_floor(skim_ctx *ctx, const float *err, int64_t rows, const int *bit_set, int n_bits,
                             double budget, uint8_t *bits_out, int64_t *total_bits)
{
    if (!ctx || !err || !bits_out) return SKIM_ERR_NULL;
    SkimBits bits;
    int rc = skim_check_bits(bit_set, n_bits, &bits);
    if (rc) return rc;
    if (rows < 1 || rows > 0x7fffffff) return SKIM_ERR_SHAPE;
    if (!(budget >= (double)bits.b_min && budget <= (double)bits.b_max)) return SKIM_ERR_BUDGET;
    const int64_t T = (int64_t)floor((double)rows * budget + 1e-6);
    int start = (int)floor(budget + 1e-9);             // every row starts at the budget rounded down
    if (start > bits.b_max) start = bits.b_max;
    const int64_t K = T - rows * (int64_t)start;
    if (K < 0 || K > rows * (int64_t)(bits.b_max - start)) return SKIM_ERR_BUDGET;
    if (total_bits) *total_bits = T;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_allocate(ctx, err, rows, bits, start - bits.b_min, K, bits_out);
}

namespace {
int optimal_plan(int64_t rows, const int *bit_set, int n_bits, double budget, SkimBits *bits, int64_t *T, int64_t *K)
{
    int rc = skim_check_bits(bit_set, n_bits, bits);
    if (rc) return rc;
    if (rows < 1 || rows > 0x7fffffff) return SKIM_ERR_SHAPE;
    if (!(budget >= (double)bits->b_min && budget <= (double)bits->b_max)) return SKIM_ERR_BUDGET;
    *T = (int64_t)floor((double)rows * budget + 1e-6);
    *K = *T - rows * (int64_t)bits->b_min;
    if (*K < 0 || *K > rows * (int64_t)(bits->b_max - bits->b_min)) return SKIM_ERR_BUDGET;
    return SKIM_OK;
}
}  // namespace

int skim_allocate_optimal_bytes(int64_t rows, const int *bit_set, int n_bits, double budget, size_t *out)
{
    if (!out) return SKIM_ERR_NULL;
    SkimBits bits;
    int64_t T, K;
    int rc = optimal_plan(rows, bit_set, n_bits, budget, &bits, &T, &K);
    if (rc) return rc;
    *out = skim_allocate_optimal_scratch(rows, K);
    return SKIM_OK;
}

int skim_allocate_optimal(skim_ctx *ctx, const float *err, int64_t rows, const int *bit_set, int n_bits, double budget,
                          void *scratch, size_t scratch_bytes, uint8_t *bits_out, int64_t *total_bits, double *cost)
{
    if (!ctx || !err || !bits_out || !scratch) return SKIM_ERR_NULL;
    SkimBits bits;
    int64_t T, K;
    int rc = optimal_plan(rows, bit_set, n_bits, budget, &bits, &T, &K);
    if (rc) return rc;
    if ((reinterpret_cast<uintptr_t>(scratch) & 255u) != 0 || scratch_bytes < skim_allocate_optimal_scratch(rows, K))
        return SKIM_ERR_WORKSPACE;
    if (total_bits) *total_bits = T;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_allocate_optimal(ctx, err, rows, bits, K, scratch, bits_out, cost);
}

int skim_packed_layout(int64_t rows, int64_t cols, const int *bit_set, int n_bits, int64_t *row_stride_words,
                       size_t *max_packed_bytes)
{
    SkimBits bits;
    int rc = skim_check_bits(bit_set, n_bits, &bits);
    if (rc) return rc;
    if (rows < 0 || cols < 1) return SKIM_ERR_SHAPE;
    if (row_stride_words)
        for (int b = 0; b < n_bits; ++b) row_stride_words[b] = skim_row_stride_words(cols, bit_set[b]);
    if (max_packed_bytes) *max_packed_bytes = (size_t)rows * (size_t)skim_row_stride_words(cols, bits.b_max) * 4;
    return SKIM_OK;
}

int skim_quantize(skim_ctx *ctx, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld, const uint8_t *bits,
                  const float *centroids, const int *bit_set, int n_bits, uint32_t *packed, int32_t *row_order,
                  int64_t *group_info, uint16_t *lut)
{
    if (!ctx || !W || !bits || !centroids || !packed || !row_order || !group_info || !lut) return SKIM_ERR_NULL;
    SkimBits bs;
    int rc = skim_check_bits(bit_set, n_bits, &bs);
    if (rc) return rc;
    rc = check_matrix(ctx, rows, cols, ld);
    if (rc) return rc;
    if (rows < 1) return SKIM_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(packed) & 15u) != 0) return SKIM_ERR_ALIGN;
    rc = check_workspace(ctx, rows, cols);
    if (rc) return rc;
    if (ctx->scaled && ctx->scale_cols != cols) return SKIM_ERR_SCALE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_quantize(ctx, W, rows, cols, ld, bits, centroids, bs, packed, row_order, group_info, lut);
}

namespace {
int check_unpack(const skim_ctx *ctx, int64_t rows, int64_t cols)
{
    if (rows < 0 || rows > 0x7fffffff || cols < 1 || cols > 0x7fffff00) return SKIM_ERR_SHAPE;
    // the per-column vector of one block lives in shared memory
    if ((size_t)((cols + 255) / 256 * 256) * sizeof(float) > (size_t)ctx->max_smem_optin) return SKIM_ERR_SHAPE;
    return SKIM_OK;
}
}  // namespace

int skim_dequantize(skim_ctx *ctx, const uint32_t *packed, const int32_t *row_order, const int64_t *group_info,
                    const uint16_t *lut, const float *s, int64_t rows, int64_t cols, const int *bit_set, int n_bits,
                    uint16_t *out, int64_t ld_out)
{
    if (!ctx || !packed || !row_order || !group_info || !lut || !out) return SKIM_ERR_NULL;
    SkimBits bs;
    int rc = skim_check_bits(bit_set, n_bits, &bs);
    if (rc) return rc;
    rc = check_unpack(ctx, rows, cols);
    if (rc) return rc;
    if (ld_out < cols) return SKIM_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_dequantize(ctx, packed, row_order, group_info, lut, s, rows, cols, bs, out, ld_out);
}

int skim_matvec(skim_ctx *ctx, const uint32_t *packed, const int32_t *row_order, const int64_t *group_info,
                const uint16_t *lut, const float *s, const uint16_t *x, int64_t rows, int64_t cols,
                const int *bit_set, int n_bits, float *y)
{
    if (!ctx || !packed || !row_order || !group_info || !lut || !x || !y) return SKIM_ERR_NULL;
    SkimBits bs;
    int rc = skim_check_bits(bit_set, n_bits, &bs);
    if (rc) return rc;
    rc = check_unpack(ctx, rows, cols);
    if (rc) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_matvec(ctx, packed, row_order, group_info, lut, s, x, rows, cols, bs, y);
}

int skim_scale_update(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                      int64_t ld, const uint8_t *labels, float *alpha, int steps, float lr0, float decay,
                      int decay_every, double *loss_trace)
{
    if (!ctx || !W || !importance || !labels || !alpha) return SKIM_ERR_NULL;
    int rc = check_matrix(ctx, rows, cols, ld);
    if (rc) return rc;
    if (rows < 1 || steps < 0 || decay_every < 1 || !(lr0 > 0.0f) || !(decay > 0.0f)) return SKIM_ERR_SHAPE;
    rc = check_workspace(ctx, rows, cols);
    if (rc) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_scale_update(ctx, W, importance, rows, cols, ld, labels, alpha, steps, lr0, decay, decay_every,
                                    loss_trace);
}

int skim_residual(skim_ctx *ctx, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld, const float *centroids,
                  const uint8_t *row_bits, int width, const int *bit_set, int n_bits, const float *s, int exp2,
                  uint16_t *D, int64_t ldd)
{
    if (!ctx || !W || !centroids || !D) return SKIM_ERR_NULL;
    SkimBits bs;
    int rc = skim_check_bits(bit_set, n_bits, &bs);
    if (rc) return rc;
    if (rows < 0 || rows > 0x7fffffff || cols < 1 || cols > 0x7fffff00 || ld < cols || ldd < cols) return SKIM_ERR_SHAPE;
    if (exp2 < 0 || exp2 > 24) return SKIM_ERR_SHAPE;
    if (!row_bits && (width < bs.b_min || width > bs.b_max)) return SKIM_ERR_BITSET;
    rc = check_workspace(ctx, rows, cols);
    if (rc) return rc;
    if ((s != nullptr) != ctx->scaled || (ctx->scaled && ctx->scale_cols != cols)) return SKIM_ERR_SCALE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_residual(ctx, W, rows, cols, ld, centroids, row_bits, width, bs, s, exp2, D, ldd);
}

int skim_err_lfull_bytes(int64_t rows, int64_t cols, size_t *out)
{
    if (!out) return SKIM_ERR_NULL;
    if (rows < 0 || rows > 0x7fffff00 || cols < 8 || cols > 0x7fffff00) return SKIM_ERR_SHAPE;
    *out = skim_lfull_scratch_bytes(rows, cols);
    return SKIM_OK;
}

int skim_err_lfull(skim_ctx *ctx, const uint16_t *D, int64_t rows, int64_t cols, int64_t ldd, const uint16_t *H,
                   int64_t ldh, int exp2, void *scratch, size_t scratch_bytes, float *err, int64_t err_stride)
{
    if (!ctx || !D || !H || !scratch || !err) return SKIM_ERR_NULL;
    if (rows < 0 || rows > 0x7fffff00 || cols < 8 || cols > 0x7fffff00 || (cols % 8) != 0) return SKIM_ERR_SHAPE;
    if (ldd < cols || ldh < cols || (ldd % 8) != 0 || (ldh % 8) != 0 || err_stride < 1) return SKIM_ERR_SHAPE;
    if (exp2 < 0 || exp2 > 24) return SKIM_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(D) & 15u) || (reinterpret_cast<uintptr_t>(H) & 15u)) return SKIM_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(scratch) & 255u) != 0 || scratch_bytes < skim_lfull_scratch_bytes(rows, cols))
        return SKIM_ERR_WORKSPACE;
    if (!ctx->ws) return SKIM_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_err_lfull(ctx, D, rows, cols, ldd, H, ldh, exp2, scratch, err, err_stride);
}

int skim_scale_lfull_bytes(int64_t rows, int64_t cols, size_t *out)
{
    if (!out) return SKIM_ERR_NULL;
    if (rows < 1 || rows > 0x7fffff00 || cols < 8 || cols > 0x7fffff00) return SKIM_ERR_SHAPE;
    *out = skim_scale_lfull_scratch_bytes(rows, cols);
    return SKIM_OK;
}

int skim_scale_update_lfull(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                            int64_t ld, const uint8_t *labels, const uint16_t *H, int64_t ldh, float *alpha, int steps,
                            float lr0, float decay, int decay_every, int exp2, void *scratch, size_t scratch_bytes,
                            double *loss_trace)
{
    if (!ctx || !W || !importance || !labels || !H || !alpha || !scratch) return SKIM_ERR_NULL;
    int rc = check_matrix(ctx, rows, cols, ld);
    if (rc) return rc;
    if (rows < 1 || steps < 0 || decay_every < 1 || !(lr0 > 0.0f) || !(decay > 0.0f)) return SKIM_ERR_SHAPE;
    if ((cols % 8) != 0 || (ld % 8) != 0 || ldh < cols || (ldh % 8) != 0 || exp2 < 0 || exp2 > 24) return SKIM_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(W) & 15u) || (reinterpret_cast<uintptr_t>(importance) & 15u) ||
        (reinterpret_cast<uintptr_t>(labels) & 15u) || (reinterpret_cast<uintptr_t>(H) & 15u))
        return SKIM_ERR_ALIGN;
    rc = check_workspace(ctx, rows, cols);
    if (rc) return rc;
    if ((reinterpret_cast<uintptr_t>(scratch) & 255u) != 0 || scratch_bytes < skim_scale_lfull_scratch_bytes(rows, cols))
        return SKIM_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    return skim_launch_scale_update_lfull(ctx, W, importance, rows, cols, ld, labels, H, ldh, alpha, steps, lr0, decay,
                                          decay_every, exp2, scratch, loss_trace);
}

// ---------------------------------------------------------------- host-buffer path

namespace {
struct Staging {
    uint16_t *W;
    float *G;
    float *centroids;
    float *err;
    uint8_t *bits;
    uint32_t *packed;
    int32_t *row_order;
    int64_t *group_info;
    uint16_t *lut;
    size_t bytes;
};

Staging carve_staging(void *base, int64_t rows, int64_t cols, const SkimBits &bs)
{
    Staging s;
    char *p = (char *)base;
    size_t off = 0;
    auto take = [&](size_t b) { char *q = p ? p + off : nullptr; off += skim_align256(b); return q; };
    s.W = (uint16_t *)take((size_t)rows * cols * 2);
    s.G = (float *)take((size_t)rows * cols * 4);
    s.centroids = (float *)take((size_t)rows * bs.sumk * 4);
    s.err = (float *)take((size_t)rows * bs.n_bits * 4);
    s.bits = (uint8_t *)take((size_t)rows);
    s.packed = (uint32_t *)take((size_t)rows * (size_t)skim_row_stride_words(cols, bs.b_max) * 4);
    s.row_order = (int32_t *)take((size_t)rows * 4);
    s.group_info = (int64_t *)take((size_t)(2 * (bs.n_bits + 1)) * 8);
    s.lut = (uint16_t *)take((size_t)rows * (size_t)(1 << bs.b_max) * 2);
    s.bytes = off;
    return s;
}
}  // namespace

int skim_host_staging_bytes(int64_t rows, int64_t cols, const int *bit_set, int n_bits, size_t *out)
{
    if (!out) return SKIM_ERR_NULL;
    SkimBits bs;
    int rc = skim_check_bits(bit_set, n_bits, &bs);
    if (rc) return rc;
    if (rows < 1 || cols < 1) return SKIM_ERR_SHAPE;
    *out = carve_staging(nullptr, rows, cols, bs).bytes;
    return SKIM_OK;
}

int skim_quantize_matrix_host(skim_ctx *ctx, const uint16_t *W_host, const float *importance_host, int64_t rows,
                              int64_t cols, const int *bit_set, int n_bits, int iters, double budget, void *staging,
                              size_t staging_bytes, float *err_host, uint8_t *bits_host, uint32_t *packed_host,
                              int32_t *row_order_host, int64_t *group_info_host, uint16_t *lut_host)
{
    if (!ctx || !W_host || !importance_host || !staging) return SKIM_ERR_NULL;
    SkimBits bs;
    int rc = skim_check_bits(bit_set, n_bits, &bs);
    if (rc) return rc;
    if (rows < 1 || cols < 1) return SKIM_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(staging) & 255u) != 0) return SKIM_ERR_WORKSPACE;
    const Staging s = carve_staging(staging, rows, cols, bs);
    if (s.bytes > staging_bytes) return SKIM_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    cudaStream_t st = ctx->stream;
    if (!ctx->copy_ready) {
        SKIM_CUDA_OK(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
        for (int k = 0; k < SKIM_HOST_CHUNKS; ++k)
            SKIM_CUDA_OK(cudaEventCreateWithFlags(&ctx->copy_done[k], cudaEventDisableTiming));
        SKIM_CUDA_OK(cudaEventCreateWithFlags(&ctx->main_idle, cudaEventDisableTiming));
        ctx->copy_ready = true;
    }
    // the staging area may still be read by earlier work on the main stream
    SKIM_CUDA_OK(cudaEventRecord(ctx->main_idle, st));
    SKIM_CUDA_OK(cudaStreamWaitEvent(ctx->copy_stream, ctx->main_idle, 0));
    // rows travel in chunks: chunk k is clustered while chunk k+1 is still on the bus
    const int64_t per = (rows + SKIM_HOST_CHUNKS - 1) / SKIM_HOST_CHUNKS;
    const int64_t chunk = per < 256 ? (rows < 256 ? rows : 256) : per;
    int k = 0;
    for (int64_t r0 = 0; r0 < rows; r0 += chunk, ++k) {
        const int64_t n = rows - r0 < chunk ? rows - r0 : chunk;
        SKIM_CUDA_OK(cudaMemcpyAsync(s.W + r0 * cols, W_host + r0 * cols, (size_t)n * cols * 2, cudaMemcpyHostToDevice,
                                     ctx->copy_stream));
        SKIM_CUDA_OK(cudaMemcpyAsync(s.G + r0 * cols, importance_host + r0 * cols, (size_t)n * cols * 4,
                                     cudaMemcpyHostToDevice, ctx->copy_stream));
        SKIM_CUDA_OK(cudaEventRecord(ctx->copy_done[k], ctx->copy_stream));
        SKIM_CUDA_OK(cudaStreamWaitEvent(st, ctx->copy_done[k], 0));
        rc = skim_cluster_rows(ctx, s.W + r0 * cols, s.G + r0 * cols, n, cols, cols, bit_set, n_bits, iters,
                               s.centroids + r0 * bs.sumk, nullptr, s.err + r0 * n_bits);
        if (rc) return rc;
    }
    rc = skim_allocate_bits(ctx, s.err, rows, bit_set, n_bits, budget, s.bits, nullptr);
    if (rc) return rc;
    rc = skim_quantize(ctx, s.W, rows, cols, cols, s.bits, s.centroids, bit_set, n_bits, s.packed, s.row_order,
                       s.group_info, s.lut);
    if (rc) return rc;
    if (err_host) SKIM_CUDA_OK(cudaMemcpyAsync(err_host, s.err, (size_t)rows * n_bits * 4, cudaMemcpyDeviceToHost, st));
    if (bits_host) SKIM_CUDA_OK(cudaMemcpyAsync(bits_host, s.bits, (size_t)rows, cudaMemcpyDeviceToHost, st));
    if (row_order_host) SKIM_CUDA_OK(cudaMemcpyAsync(row_order_host, s.row_order, (size_t)rows * 4, cudaMemcpyDeviceToHost, st));
    if (lut_host)
        SKIM_CUDA_OK(cudaMemcpyAsync(lut_host, s.lut, (size_t)rows * (size_t)(1 << bs.b_max) * 2, cudaMemcpyDeviceToHost, st));
    int64_t info[2 * (SKIM_MAX_NBITS + 1)];
    SKIM_CUDA_OK(cudaMemcpyAsync(info, s.group_info, (size_t)(2 * (n_bits + 1)) * 8, cudaMemcpyDeviceToHost, st));
    SKIM_CUDA_OK(cudaStreamSynchronize(st));
    if (group_info_host)
        for (int u = 0; u < 2 * (n_bits + 1); ++u) group_info_host[u] = info[u];
    if (packed_host) {
        // only the words the allocation really uses travel back
        const size_t words = (size_t)info[2 * n_bits + 1];
        SKIM_CUDA_OK(cudaMemcpyAsync(packed_host, s.packed, words * 4, cudaMemcpyDeviceToHost, st));
        SKIM_CUDA_OK(cudaStreamSynchronize(st));
    }
    return SKIM_OK;
}

int skim_get_status(skim_ctx *ctx, uint64_t *flags)
{
    if (!ctx) return SKIM_ERR_NULL;
    if (!ctx->ws) return SKIM_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    unsigned long long v = 0;
    SKIM_CUDA_OK(cudaMemcpyAsync(&v, ctx->ws, 8, cudaMemcpyDeviceToHost, ctx->stream));
    SKIM_CUDA_OK(cudaMemsetAsync(ctx->ws, 0, 8, ctx->stream));
    SKIM_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    if (flags) *flags = (uint64_t)v;
    return v ? SKIM_ERR_BAD_DATA : SKIM_OK;
}

int64_t skim_launch_count(const skim_ctx *ctx) { return ctx ? ctx->launches : 0; }

int skim_kernel_timing(skim_ctx *ctx, int enable)
{
    if (!ctx) return SKIM_ERR_NULL;
    if (enable && !ctx->timing_ready) {
        DeviceGuard guard(ctx->device);
        if (!guard.ok) return SKIM_ERR_CUDA;
        for (int k = 0; k < SKIM_TIMING_SLOTS; ++k)
            for (int e = 0; e < 3; ++e) SKIM_CUDA_OK(cudaEventCreate(&ctx->timing_ev[k][e]));
        ctx->timing_ready = true;
    }
    ctx->timing = enable != 0;
    ctx->timing_used = 0;
    return SKIM_OK;
}

int skim_kernel_times(skim_ctx *ctx, double *sort_ms, double *lloyd_ms, int64_t *chunks)
{
    if (!ctx) return SKIM_ERR_NULL;
    double s = 0.0, l = 0.0;
    if (ctx->timing_used > 0) {
        DeviceGuard guard(ctx->device);
        if (!guard.ok) return SKIM_ERR_CUDA;
        SKIM_CUDA_OK(cudaEventSynchronize(ctx->timing_ev[ctx->timing_used - 1][2]));
        for (int k = 0; k < ctx->timing_used; ++k) {
            float a = 0.0f, b = 0.0f;
            SKIM_CUDA_OK(cudaEventElapsedTime(&a, ctx->timing_ev[k][0], ctx->timing_ev[k][1]));
            SKIM_CUDA_OK(cudaEventElapsedTime(&b, ctx->timing_ev[k][1], ctx->timing_ev[k][2]));
            s += a;
            l += b;
        }
    }
    if (sort_ms) *sort_ms = s;
    if (lloyd_ms) *lloyd_ms = l;
    if (chunks) *chunks = ctx->timing_used;
    return SKIM_OK;
}

int skim_early_exit(skim_ctx *ctx, int enable)
{
    if (!ctx) return SKIM_ERR_NULL;
    ctx->early_exit = enable != 0;
    return SKIM_OK;
}

int skim_lloyd_iterations(skim_ctx *ctx, int64_t *iterations, int64_t *rows)
{
    if (!ctx) return SKIM_ERR_NULL;
    if (!ctx->ws) return SKIM_ERR_WORKSPACE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return SKIM_ERR_CUDA;
    unsigned long long v[2] = {0ull, 0ull};
    unsigned char *p = (unsigned char *)ctx->ws + 8;
    SKIM_CUDA_OK(cudaMemcpyAsync(v, p, 16, cudaMemcpyDeviceToHost, ctx->stream));
    SKIM_CUDA_OK(cudaMemsetAsync(p, 0, 16, ctx->stream));
    SKIM_CUDA_OK(cudaStreamSynchronize(ctx->stream));
    if (iterations) *iterations = (int64_t)v[0];
    if (rows) *rows = (int64_t)v[1];
    return SKIM_OK;
}

const char *skim_strerror(int code)
{
    switch (code) {
    case SKIM_OK: return "ok";
    case SKIM_ERR_NULL: return "a required pointer is NULL";
    case SKIM_ERR_SHAPE: return "rows, cols, ld, iters or steps out of range";
    case SKIM_ERR_BITSET: return "bit_set must be consecutive ascending widths inside [1, 4]";
    case SKIM_ERR_BUDGET: return "budget outside [b_min, b_max]";
    case SKIM_ERR_WORKSPACE: return "workspace missing, too small or misaligned";
    case SKIM_ERR_CUDA: return "a CUDA runtime call failed";
    case SKIM_ERR_BAD_DATA: return "bad data: NaN/Inf weight, negative importance, non-positive scale or width outside bit_set";
    case SKIM_ERR_SCALE: return "installed scale vector length differs from cols";
    case SKIM_ERR_ALIGN: return "output pointer not aligned as documented";
    case SKIM_ERR_STATIC_LIMIT: return "skim_quantize_static: rows exceed SKIM_STATIC_MAX_ROWS (65536), the size of the built-in scratch array";
    default: return "unknown error";
    }
}

}  // extern "C"
