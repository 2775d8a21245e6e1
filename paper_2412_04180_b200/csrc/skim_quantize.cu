// Final labels, packing and codebooks (SKIM Algorithm 3, second row loop; Section 4.2: rows of
// equal width are gathered and packed together), plus the reciprocal of the scaling vector
// (Section 4.3).
//
//   skim_rank_rows_kernel  one block: stable partition of the rows by width -> packed position of
//                          every row, row order, group starts and word offsets.
//   skim_pack_kernel       one block per row: label = number of midpoints below the element
//                          (packed fp16 compares, two weights per instruction, when no scale is
//                          installed; a 4-step search in binary32 otherwise); a thread packs whole
//                          groups of 32 elements into their b words.
#include "skim_internal.cuh"

namespace {

constexpr int RT = 1024;

__global__ void __launch_bounds__(RT) skim_rank_rows_kernel(const uint8_t *__restrict__ bits, int64_t n, int64_t cols,
                                                             int nb, int bmin, int32_t *__restrict__ row_pos,
                                                             int32_t *__restrict__ row_order,
                                                             long long *__restrict__ group_info,
                                                             unsigned long long *status)
{
    __shared__ int wsum[RT / 32][SKIM_MAX_NBITS];
    __shared__ int gstart[SKIM_MAX_NBITS + 1];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t per = (n + RT - 1) / RT;
    const int64_t r0 = min(n, (int64_t)tid * per), r1 = min(n, r0 + per);
    int cnt[SKIM_MAX_NBITS] = {0, 0, 0, 0};
    bool bad = false;
    for (int64_t i = r0; i < r1; ++i) {
        const int u = (int)bits[i] - bmin;
        if (u < 0 || u >= nb) { bad = true; continue; }
#pragma unroll
        for (int v = 0; v < SKIM_MAX_NBITS; ++v) cnt[v] += (u == v) ? 1 : 0;
    }
    if (bad) atomicOr(status, 8ull);
    int inc[SKIM_MAX_NBITS];
#pragma unroll
    for (int v = 0; v < SKIM_MAX_NBITS; ++v) inc[v] = cnt[v];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
#pragma unroll
        for (int v = 0; v < SKIM_MAX_NBITS; ++v) {
            const int t = __shfl_up_sync(0xffffffffu, inc[v], off);
            if (lane >= off) inc[v] += t;
        }
    }
    if (lane == 31) {
#pragma unroll
        for (int v = 0; v < SKIM_MAX_NBITS; ++v) wsum[warp][v] = inc[v];
    }
    __syncthreads();
    // warp 0 turns the warps' sums into exclusive prefixes; its last lane then holds the totals and lays out the groups
    if (warp == 0) {
        int x[SKIM_MAX_NBITS], run[SKIM_MAX_NBITS];
#pragma unroll
        for (int v = 0; v < SKIM_MAX_NBITS; ++v) { x[v] = wsum[lane][v]; run[v] = x[v]; }
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
#pragma unroll
            for (int v = 0; v < SKIM_MAX_NBITS; ++v) {
                const int t = __shfl_up_sync(0xffffffffu, run[v], off);
                if (lane >= off) run[v] += t;
            }
        }
#pragma unroll
        for (int v = 0; v < SKIM_MAX_NBITS; ++v) wsum[lane][v] = run[v] - x[v];
        if (lane == 31) {
            long long start = 0, word = 0;
#pragma unroll
            for (int v = 0; v < SKIM_MAX_NBITS; ++v) {
                if (v < nb) {
                    gstart[v] = (int)start;
                    group_info[v] = start;
                    group_info[nb + 1 + v] = word;
                    start += run[v];
                    word += (long long)run[v] * skim_row_stride_words(cols, bmin + v);
                }
            }
            gstart[nb] = (int)start;
            group_info[nb] = start;
            group_info[2 * nb + 1] = word;
        }
    }
    __syncthreads();
    int before[SKIM_MAX_NBITS];
#pragma unroll
    for (int v = 0; v < SKIM_MAX_NBITS; ++v) before[v] = inc[v] - cnt[v] + wsum[warp][v];
    for (int64_t i = r0; i < r1; ++i) {
        const int u = (int)bits[i] - bmin;
        if (u < 0 || u >= nb) { row_pos[i] = -1; continue; }
        int pos = 0;
#pragma unroll
        for (int v = 0; v < SKIM_MAX_NBITS; ++v) {
            if (u == v) { pos = gstart[v] + before[v]; before[v] += 1; }
        }
        row_pos[i] = pos;
        row_order[pos] = (int32_t)i;
    }
}


struct PackArgs {
    const uint16_t *W;
    const float *rscale;
    const uint8_t *bits;
    const float *centroids;
    const int32_t *row_pos;
    const long long *group_info;
    int64_t ld;
    int cols;
    int nb, bmin, sumk;
    int vec_ok;   // rows start 16-byte aligned: 128-bit loads allowed
    uint32_t *packed;
    uint16_t *lut;
};

// Labels of 8 fp16 weights (no scale installed) with packed half-precision compares: a weight is
// above a boundary exactly when it is above the boundary rounded down to fp16, so two weights are
// compared per instruction and the label is the running sum of the 0/1 results.  Returns the 8
// labels as B-bit fields.
template <int B>
__device__ __forceinline__ uint32_t labels8_half(const uint4 raw, const __half2 *th)
{
    const __half2 *p = reinterpret_cast<const __half2 *>(&raw);
    const __half2 magic = __floats2half2_rn(1024.0f, 1024.0f);   // 1024 + n has n in its low mantissa bits
    uint32_t v = 0;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        __half2 cnt = magic;
#pragma unroll
        for (int j = 0; j < (1 << B) - 1; ++j) cnt = __hadd2(cnt, __hgt2(p[u], th[j]));
        const uint32_t bits = *reinterpret_cast<const uint32_t *>(&cnt);
        v |= (bits & 0xfu) << ((2 * u) * B);
        v |= ((bits >> 16) & 0xfu) << ((2 * u + 1) * B);
    }
    return v;
}

// Eight blocks of this size are resident per SM at 64 registers.  A block lives for little more than the two round
// trips of its parameter loads, so many small resident blocks hide them better than few large ones (measured: 64,
// 128, 192, 256 and 384 threads give 42.9, 40.0, 43.5, 44.3 and 45.8 us for rank + pack of 4096 x 11008).
constexpr int PACK_MAX_THREADS = 128;

// Labels of 8 elements starting at e0 on the general path (a scale vector installed, unaligned rows, or the ragged
// end of a row): the clustered value in binary32, then a 4-step search of the binary32 thresholds.
template <int B>
__device__ __forceinline__ uint32_t labels8_general(const PackArgs &a, const uint16_t *Wr, int e0, const float *tf)
{
    float x[8];
    if (a.vec_ok && e0 + 8 <= a.cols) {
        const uint4 raw = *reinterpret_cast<const uint4 *>(Wr + e0);
        const __half2 *h2 = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float2 f = __half22float2(h2[u]);
            x[2 * u] = f.x;
            x[2 * u + 1] = f.y;
        }
        if (a.rscale) {
            const float4 r0 = *reinterpret_cast<const float4 *>(a.rscale + e0);
            const float4 r1 = *reinterpret_cast<const float4 *>(a.rscale + e0 + 4);
            x[0] = __fmul_rn(x[0], r0.x); x[1] = __fmul_rn(x[1], r0.y);
            x[2] = __fmul_rn(x[2], r0.z); x[3] = __fmul_rn(x[3], r0.w);
            x[4] = __fmul_rn(x[4], r1.x); x[5] = __fmul_rn(x[5], r1.y);
            x[6] = __fmul_rn(x[6], r1.z); x[7] = __fmul_rn(x[7], r1.w);
        }
    } else {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int e = e0 + u;
            float xv = -__int_as_float(0x7f800000);    // past the row: label 0 (zero padding)
            if (e < a.cols) {
                xv = __half2float(__ushort_as_half(Wr[e]));
                if (a.rscale) xv = __fmul_rn(xv, a.rscale[e]);
            }
            x[u] = xv;
        }
    }
    uint32_t v = 0;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        int code = (x[u] > tf[7]) ? 8 : 0;
        code += (x[u] > tf[code + 3]) ? 4 : 0;
        code += (x[u] > tf[code + 1]) ? 2 : 0;
        code += (x[u] > tf[code]) ? 1 : 0;
        v |= (uint32_t)code << (u * B);
    }
    return v;
}

// One row at width B: a thread packs whole groups of 32 elements into their B words -- four 128-bit loads, the
// labels of 8 elements at a time, the four 8B-bit fields joined with compile-time shifts -- so that no bits cross
// threads (an earlier version gave a thread 8 elements and merged four threads' fields with 64-bit shuffles, which
// cost more instructions than the compares).
template <int B>
__device__ __forceinline__ void pack_row(const PackArgs &a, const uint16_t *Wr, const __half2 *th, const float *tf,
                                         uint32_t *dst, int64_t stride, bool fast, uint4 (&raw)[4])
{
    const int ngroups = (int)((stride + B - 1) / B);    // a group: 32 elements -> B words
    // `raw` arrives holding the weights of the thread's first group (requested before the row's parameters were)
    for (int grp = threadIdx.x; grp < ngroups; grp += blockDim.x) {
        const int e0 = grp * 32;
        uint32_t v[4];
        if (fast && e0 + 32 <= a.cols) {
            if (grp != (int)threadIdx.x) {
#pragma unroll
                for (int q = 0; q < 4; ++q) raw[q] = __ldg(reinterpret_cast<const uint4 *>(Wr + e0 + 8 * q));
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = labels8_half<B>(raw[q], th);
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = labels8_general<B>(a, Wr, e0 + 8 * q, tf);
        }
        uint32_t word[4] = {0u, 0u, 0u, 0u};
        if constexpr (B == 4) {
            word[0] = v[0]; word[1] = v[1]; word[2] = v[2]; word[3] = v[3];
        } else if constexpr (B == 3) {
            word[0] = v[0] | (v[1] << 24);
            word[1] = (v[1] >> 8) | (v[2] << 16);
            word[2] = (v[2] >> 16) | (v[3] << 8);
        } else if constexpr (B == 2) {
            word[0] = v[0] | (v[1] << 16);
            word[1] = v[2] | (v[3] << 16);
        } else {
            word[0] = v[0] | (v[1] << 8) | (v[2] << 16) | (v[3] << 24);
        }
        const int64_t w0 = (int64_t)grp * B;
        if (B == 4 && w0 + 4 <= stride) {
            *reinterpret_cast<uint4 *>(dst + w0) = make_uint4(word[0], word[1], word[2], word[3]);   // rows start 16-byte aligned
        } else {
#pragma unroll
            for (int w = 0; w < B; ++w)
                if (w0 + w < stride) dst[w0 + w] = word[w];
        }
    }
}

__global__ void __launch_bounds__(PACK_MAX_THREADS, 8) skim_pack_kernel(PackArgs a)
{
    __shared__ float tf[16];
    __shared__ __half2 th_s[16];
    const int tid = threadIdx.x;
    const int64_t row = blockIdx.x;
    const uint16_t *Wr = a.W + row * a.ld;
    const bool fast = a.vec_ok && !a.rscale;
    // the weights of the thread's first group and the row's two parameters are requested together; the codebook
    // and the thresholds need the width, so they are one more round trip
    uint4 raw[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) raw[q] = make_uint4(0u, 0u, 0u, 0u);
    if (fast && tid * 32 + 32 <= a.cols) {
#pragma unroll
        for (int q = 0; q < 4; ++q) raw[q] = __ldg(reinterpret_cast<const uint4 *>(Wr + tid * 32 + 8 * q));
    }
    const int pos = a.row_pos[row];
    const int b = (int)a.bits[row];
    if (pos < 0) return;
    const int bi = b - a.bmin;
    const int k = 1 << b;
    const int off = (1 << a.bmin) * ((1 << bi) - 1);
    const int kmax = 1 << (a.bmin + a.nb - 1);
    const float *c = a.centroids + row * a.sumk + off;
    if (tid < 16) {
        const float cj = c[min(tid, k - 1)];
        if (tid < kmax) a.lut[row * kmax + tid] = __half_as_ushort(__float2half_rn(cj));
        float t = __int_as_float(0x7f800000);
        if (tid < k - 1) {
            t = __double2float_rd(0.5 * ((double)cj + (double)c[tid + 1]));
            if (t == 0.0f) t = 0.0f;
        }
        tf[tid] = t;
        th_s[tid] = __half2half2(__float2half_rd(t));
    }
    __syncthreads();
    __half2 th[15];
#pragma unroll
    for (int j = 0; j < 15; ++j) th[j] = th_s[j];
    const int64_t stride = skim_row_stride_words(a.cols, b);
    uint32_t *dst = a.packed + a.group_info[a.nb + 1 + bi] + (int64_t)(pos - a.group_info[bi]) * stride;
    switch (b) {
    case 1: pack_row<1>(a, Wr, th, tf, dst, stride, fast, raw); break;
    case 2: pack_row<2>(a, Wr, th, tf, dst, stride, fast, raw); break;
    case 3: pack_row<3>(a, Wr, th, tf, dst, stride, fast, raw); break;
    default: pack_row<4>(a, Wr, th, tf, dst, stride, fast, raw); break;
    }
}

// Threads of a pack block: one per group of 32 elements of the longest packed row, in whole warps, at most
// PACK_MAX_THREADS (longer rows take several groups per thread).
static unsigned pack_threads(int64_t cols, const SkimBits &bs)
{
    int64_t most = 1;
    for (int u = 0; u < bs.n_bits; ++u) {
        const int b = bs.b_min + u;
        const int64_t g = (skim_row_stride_words(cols, b) + b - 1) / b;
        if (g > most) most = g;
    }
    const int64_t t = (most + 31) / 32 * 32;
    return (unsigned)(t > PACK_MAX_THREADS ? PACK_MAX_THREADS : t);
}

__global__ void skim_reciprocal_kernel(const float *__restrict__ s, int64_t cols, float *__restrict__ r,
                                       unsigned long long *status)
{
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= cols) return;
    const float v = s[j];
    if (!(v > 0.0f) || v > 3.0e38f) atomicOr(status, (unsigned long long)SKIM_STATUS_BAD_SCALE);
    r[j] = __fdiv_rn(1.0f, v);
}

}  // namespace

int skim_launch_reciprocal(skim_ctx *ctx, const float *s, int64_t cols)
{
    SkimWorkspace ws = skim_carve(ctx->ws, 0, cols);
    const int threads = 256;
    const unsigned blocks = (unsigned)((cols + threads - 1) / threads);
    skim_reciprocal_kernel<<<blocks, threads, 0, ctx->stream>>>(s, cols, ws.rscale, ws.status);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}

int skim_launch_quantize(skim_ctx *ctx, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld,
                         const uint8_t *bits, const float *centroids, const SkimBits &bs, uint32_t *packed,
                         int32_t *row_order, int64_t *group_info, uint16_t *lut)
{
    SkimWorkspace ws = skim_carve(ctx->ws, rows, cols);
    skim_rank_rows_kernel<<<1, RT, 0, ctx->stream>>>(bits, rows, cols, bs.n_bits, bs.b_min, ws.row_pos, row_order,
                                                     (long long *)group_info, ws.status);
    SKIM_CUDA_OK(cudaGetLastError());
    PackArgs a;
    a.W = W;
    a.rscale = ctx->scaled ? ws.rscale : nullptr;
    a.bits = bits;
    a.centroids = centroids;
    a.row_pos = ws.row_pos;
    a.group_info = (const long long *)group_info;
    a.ld = ld;
    a.cols = (int)cols;
    a.nb = bs.n_bits;
    a.bmin = bs.b_min;
    a.sumk = bs.sumk;
    a.vec_ok = ((reinterpret_cast<uintptr_t>(W) & 15u) == 0 && (ld % 8) == 0) ? 1 : 0;
    a.packed = packed;
    a.lut = lut;
    skim_pack_kernel<<<(unsigned)rows, pack_threads(cols, bs), 0, ctx->stream>>>(a);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 2;
    return SKIM_OK;
}

// ---------------------------------------------------------------- entry point that allocates nothing
//
// skim_quantize_static is skim_quantize for callers that cannot provide a workspace because they
// may not allocate device memory at all: code running inside a region where cudaMalloc is
// forbidden or would deadlock (an allocator callback, a real-time loop with a fixed memory plan,
// a plugin that only borrows its host's buffers).  Its scratch (the per-row packed position and a
// status word) lives in a fixed array inside the library image instead of a caller workspace.

#include <mutex>

#define SKIM_STATIC_SCRATCH_BYTES (256 + (size_t)SKIM_STATIC_MAX_ROWS * 4)

// Resident on every GPU that loads the library, until the process exits.
static __device__ __align__(256) unsigned char skim_static_scratch[SKIM_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device.  In host code the array's name is
// only a handle, so the address has to be asked for, once per device, with that device current.
int static_scratch_address(void **out)
{
    int dev = -1;
    SKIM_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SKIM_ERR_SHAPE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        SKIM_CUDA_OK(cudaGetSymbolAddress(&p, skim_static_scratch));
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return SKIM_OK;
}
}  // namespace

extern "C" int skim_quantize_static(void *cuda_stream, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld,
                                    const uint8_t *bits, const float *centroids, const int *bit_set, int n_bits,
                                    uint32_t *packed, int32_t *row_order, int64_t *group_info, uint16_t *lut)
{
    if (!W || !bits || !centroids || !packed || !row_order || !group_info || !lut) return SKIM_ERR_NULL;
    SkimBits bs;
    int rc = skim_check_bits(bit_set, n_bits, &bs);
    if (rc) return rc;
    if (rows < 1 || cols < 1 || cols > 0x7fffffff / 8 || ld < cols) return SKIM_ERR_SHAPE;
    if (rows > SKIM_STATIC_MAX_ROWS) return SKIM_ERR_STATIC_LIMIT;
    if ((reinterpret_cast<uintptr_t>(packed) & 15u) != 0) return SKIM_ERR_ALIGN;
    void *scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc) return rc;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long *status = (unsigned long long *)scratch;
    int32_t *row_pos = (int32_t *)((unsigned char *)scratch + 256);
    // the array keeps whatever the previous call left: the status word must start at zero
    // (row_pos is rewritten for every row before it is read)
    SKIM_CUDA_OK(cudaMemsetAsync(status, 0, 256, stream));
    skim_rank_rows_kernel<<<1, RT, 0, stream>>>(bits, rows, cols, bs.n_bits, bs.b_min, row_pos, row_order,
                                                (long long *)group_info, status);
    SKIM_CUDA_OK(cudaGetLastError());
    PackArgs a;
    a.W = W;
    a.rscale = nullptr;
    a.bits = bits;
    a.centroids = centroids;
    a.row_pos = row_pos;
    a.group_info = (const long long *)group_info;
    a.ld = ld;
    a.cols = (int)cols;
    a.nb = bs.n_bits;
    a.bmin = bs.b_min;
    a.sumk = bs.sumk;
    a.vec_ok = ((reinterpret_cast<uintptr_t>(W) & 15u) == 0 && (ld % 8) == 0) ? 1 : 0;
    a.packed = packed;
    a.lut = lut;
    skim_pack_kernel<<<(unsigned)rows, pack_threads(cols, bs), 0, stream>>>(a);
    SKIM_CUDA_OK(cudaGetLastError());
    return SKIM_OK;
}
