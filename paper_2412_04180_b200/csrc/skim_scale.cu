// Scaling-vector training with the labels held fixed (SKIM Section 4.3, Algorithm 2, inner
// repeat; optimiser settings of Section 5.1).
//
//   loss(alpha) = sum_ij g_ij (W_ij - alpha_j c_{i,l_ij})^2,
//   c_ik        = sum_{j in k} g_ij W_ij / alpha_j  /  sum_{j in k} g_ij   (re-fitted each step)
//
// Per Adam step two kernels run:
//   skim_scale_rows_kernel  a fixed set of blocks, each walking a contiguous chunk of rows.  For
//       a row it makes three passes over (W, g, label): cluster sums -> centroids; residual
//       sums; gradient terms, which it adds to a per-block column accumulator in shared memory.
//       The first pass comes from HBM, the other two hit L2.  Per-thread private accumulator
//       slots in shared memory keep every sum in binary64 without atomics.
//   skim_scale_adam_kernel  sums the per-block column partials in block order (deterministic),
//       applies the Adam update to the binary64 master copy of alpha and refreshes 1/alpha.
#include "skim_internal.cuh"

namespace {

constexpr int KC = 16;  // clusters per row at most (4 bits)

struct ScaleArgs {
    const uint16_t *W;
    const float *G;
    const uint8_t *labels;
    const double *alpha;
    const double *ralpha;
    int64_t rows, ld;
    int cols;
    int rows_per_block;
    double *grad_part;   // [gridDim.x][cols]
    double *loss_part;   // [gridDim.x]
};

template <int THREADS>
__global__ void __launch_bounds__(THREADS) skim_scale_rows_kernel(ScaleArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *colacc = reinterpret_cast<double *>(smem_raw);            // [cols]
    double *acc0 = colacc + a.cols;                                   // [KC][THREADS]
    double *acc1 = acc0 + KC * THREADS;                               // [KC][THREADS]
    double *Gv = acc1 + KC * THREADS;                                 // [KC]
    double *Cv = Gv + KC;                                             // [KC]
    double *Rv = Cv + KC;                                             // [KC]
    double *red = Rv + KC;                                            // [32]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = THREADS / 32;

    for (int e = tid; e < a.cols; e += THREADS) colacc[e] = 0.0;
    double loss = 0.0;
    const int64_t r0 = (int64_t)blockIdx.x * a.rows_per_block;
    const int64_t r1 = min(a.rows, r0 + a.rows_per_block);
    for (int64_t row = r0; row < r1; ++row) {
        const uint16_t *Wr = a.W + row * a.ld;
        const float *Gr = a.G + row * a.ld;
        const uint8_t *Lr = a.labels + row * (int64_t)a.cols;
#pragma unroll
        for (int k = 0; k < KC; ++k) { acc0[k * THREADS + tid] = 0.0; acc1[k * THREADS + tid] = 0.0; }
        // pass 1: G_k = sum g, S_k = sum g w / alpha
        for (int e = tid; e < a.cols; e += THREADS) {
            const int l = Lr[e] & (KC - 1);
            const double g = (double)Gr[e];
            const double w = (double)__half2float(__ushort_as_half(Wr[e]));
            acc0[l * THREADS + tid] += g;
            acc1[l * THREADS + tid] += g * w * a.ralpha[e];
        }
        __syncthreads();
        for (int k = warp; k < KC; k += NW) {
            double s0 = 0.0, s1 = 0.0;
            for (int t = lane; t < THREADS; t += 32) { s0 += acc0[k * THREADS + t]; s1 += acc1[k * THREADS + t]; }
#pragma unroll
            for (int off = 16; off; off >>= 1) {
                s0 += __shfl_xor_sync(0xffffffffu, s0, off);
                s1 += __shfl_xor_sync(0xffffffffu, s1, off);
            }
            if (lane == 0) { Gv[k] = s0; Cv[k] = s0 > 0.0 ? s1 / s0 : 0.0; }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < KC; ++k) acc0[k * THREADS + tid] = 0.0;
        // pass 2: residuals r = w - alpha c; loss; R_k = sum g r alpha
        for (int e = tid; e < a.cols; e += THREADS) {
            const int l = Lr[e] & (KC - 1);
            const double g = (double)Gr[e];
            const double w = (double)__half2float(__ushort_as_half(Wr[e]));
            const double al = a.alpha[e];
            const double r = w - al * Cv[l];
            loss = fma(g * r, r, loss);
            acc0[l * THREADS + tid] += g * r * al;
        }
        __syncthreads();
        for (int k = warp; k < KC; k += NW) {
            double s0 = 0.0;
            for (int t = lane; t < THREADS; t += 32) s0 += acc0[k * THREADS + t];
#pragma unroll
            for (int off = 16; off; off >>= 1) s0 += __shfl_xor_sync(0xffffffffu, s0, off);
            if (lane == 0) Rv[k] = s0;
        }
        __syncthreads();
        // pass 3: d loss / d alpha_j, both terms (directly, and through the re-fitted centroid)
        for (int e = tid; e < a.cols; e += THREADS) {
            const int l = Lr[e] & (KC - 1);
            const double g = (double)Gr[e];
            const double w = (double)__half2float(__ushort_as_half(Wr[e]));
            const double al = a.alpha[e], ra = a.ralpha[e];
            const double c = Cv[l];
            const double r = w - al * c;
            double d = -2.0 * g * r * c;
            if (Gv[l] > 0.0) d += 2.0 * Rv[l] * g * w * ra * ra / Gv[l];
            colacc[e] += d;
        }
        __syncthreads();
    }
    for (int e = tid; e < a.cols; e += THREADS) a.grad_part[(int64_t)blockIdx.x * a.cols + e] = colacc[e];
#pragma unroll
    for (int off = 16; off; off >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, off);
    if (lane == 0) red[warp] = loss;
    __syncthreads();
    if (tid == 0) {
        double s = 0.0;
        for (int w = 0; w < NW; ++w) s += red[w];
        a.loss_part[blockIdx.x] = s;
    }
}

__global__ void skim_scale_adam_kernel(const double *__restrict__ grad_part, const double *__restrict__ loss_part,
                                       int nblocks, int cols, double *alpha, double *ralpha, double *m1, double *m2,
                                       double lr, double beta1, double beta2, double bc1, double bc2, double eps,
                                       double *loss_out)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j == 0 && loss_out) {
        double s = 0.0;
        for (int b = 0; b < nblocks; ++b) s += loss_part[b];
        *loss_out = s;
    }
    if (j >= cols) return;
    double g = 0.0;
    for (int b = 0; b < nblocks; ++b) g += grad_part[(int64_t)b * cols + j];
    const double a1 = beta1 * m1[j] + (1.0 - beta1) * g;
    const double a2 = beta2 * m2[j] + (1.0 - beta2) * g * g;
    m1[j] = a1;
    m2[j] = a2;
    const double al = alpha[j] - lr * (a1 / bc1) / (sqrt(a2 / bc2) + eps);
    alpha[j] = al;
    ralpha[j] = 1.0 / al;
}

__global__ void skim_scale_init_kernel(const float *__restrict__ alpha32, int cols, double *alpha, double *ralpha,
                                       double *m1, double *m2, unsigned long long *status)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= cols) return;
    const float v = alpha32[j];
    if (!(v > 0.0f) || v > 3.0e38f) atomicOr(status, (unsigned long long)SKIM_STATUS_BAD_SCALE);
    alpha[j] = (double)v;
    ralpha[j] = 1.0 / (double)v;
    m1[j] = 0.0;
    m2[j] = 0.0;
}

__global__ void skim_scale_finish_kernel(const double *__restrict__ alpha, int cols, float *__restrict__ alpha32)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < cols) alpha32[j] = (float)alpha[j];
}

size_t scale_smem(int cols, int threads) { return ((size_t)cols + 2 * KC * (size_t)threads + 3 * KC + 32) * 8; }

}  // namespace

int skim_launch_scale_update(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                             int64_t ld, const uint8_t *labels, float *alpha, int steps, float lr0, float decay,
                             int decay_every, double *loss_trace)
{
    SkimWorkspace ws = skim_carve(ctx->ws, rows, cols);
    int threads = 256;
    size_t smem = scale_smem((int)cols, threads);
    if (smem > (size_t)ctx->max_smem_optin) { threads = 128; smem = scale_smem((int)cols, threads); }
    if (smem > (size_t)ctx->max_smem_optin) return SKIM_ERR_SHAPE;
    int nblocks = (int)(rows < SKIM_SCALE_MAX_CTAS ? rows : SKIM_SCALE_MAX_CTAS);
    const int per = (int)((rows + nblocks - 1) / nblocks);
    nblocks = (int)((rows + per - 1) / per);
    auto kernel = threads == 256 ? skim_scale_rows_kernel<256> : skim_scale_rows_kernel<128>;
    SKIM_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const unsigned cb = (unsigned)((cols + 255) / 256);
    skim_scale_init_kernel<<<cb, 256, 0, ctx->stream>>>(alpha, (int)cols, ws.alpha64, ws.ralpha, ws.adam_m, ws.adam_v,
                                                        ws.status);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    ScaleArgs a;
    a.W = W;
    a.G = importance;
    a.labels = labels;
    a.alpha = ws.alpha64;
    a.ralpha = ws.ralpha;
    a.rows = rows;
    a.ld = ld;
    a.cols = (int)cols;
    a.rows_per_block = per;
    a.grad_part = ws.grad_part;
    a.loss_part = ws.loss_part;
    const double beta1 = 0.9, beta2 = 0.999, eps = 1e-8;
    double p1 = 1.0, p2 = 1.0, lr = (double)lr0;
    for (int t = 0; t < steps; ++t) {
        if (t > 0 && t % decay_every == 0) lr *= (double)decay;
        p1 *= beta1;
        p2 *= beta2;
        kernel<<<nblocks, threads, smem, ctx->stream>>>(a);
        SKIM_CUDA_OK(cudaGetLastError());
        skim_scale_adam_kernel<<<cb, 256, 0, ctx->stream>>>(ws.grad_part, ws.loss_part, nblocks, (int)cols, ws.alpha64,
                                                            ws.ralpha, ws.adam_m, ws.adam_v, lr, beta1, beta2,
                                                            1.0 - p1, 1.0 - p2, eps,
                                                            loss_trace ? loss_trace + t : nullptr);
        SKIM_CUDA_OK(cudaGetLastError());
        ctx->launches += 2;
    }
    skim_scale_finish_kernel<<<cb, 256, 0, ctx->stream>>>(ws.alpha64, (int)cols, alpha);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
