// Consumers of the packed form (SKIM Section 4.2, last paragraph: rows of equal width are stored and
// processed together; Section 4 overview and Section 4.3: a dequantised weight is its codebook
// entry times the scaling vector, Wq = Quant(W * alpha^-1) * alpha):
//   skim_dequantize  packed codes + per-row codebooks (+ alpha) -> fp16 matrix in source-row order
//   skim_matvec      y = Wq x taken straight from the packed codes, never forming Wq
//
// One warp owns one packed row.  A step covers 256 consecutive elements: the warp fetches the 8b
// words that hold them with one coalesced load, every lane cuts its 8 codes out of the bit stream
// (two shuffles and a funnel shift, since 3-bit codes straddle words), looks the codebook entry up
// in the warp's 16-word copy of the row's codebook in shared memory (16 consecutive words: no bank
// conflicts, equal indices are broadcast) and meets the per-column vector (alpha, or alpha * x),
// also in shared memory, where the block put it once for all of its rows.  Both kernels are bound by HBM
// traffic: b/8 bytes per element in, and for the dequantiser 2 bytes per element out.
#include "skim_internal.cuh"

namespace {

constexpr int UT = 1024;            // threads per block: 32 rows share one copy of the column vector
constexpr int UW = UT / 32;
constexpr int STEP = 256;           // elements per warp step

struct UnpackArgs {
    const uint32_t *packed;
    const int32_t *row_order;
    const long long *group_info;    // [nb + 1] first packed row of every group, then [nb + 1] word offsets
    const uint16_t *lut;            // [rows][kmax] binary16
    const float *s;                 // [cols] or nullptr
    const uint16_t *x;              // [cols] binary16 (mat-vec only)
    int64_t rows;
    int cols;
    int nb, bmin, kmax;
    uint16_t *out;                  // dequantiser: [rows][ld]
    int64_t ld;
    int out_vec;                    // rows of `out` are 16-byte aligned
    float *y;                       // mat-vec: [rows]
};

// Packed row p: its width index, source row and first word.  False when p is not a placed row.
__device__ __forceinline__ bool locate_row(const UnpackArgs &a, int64_t p, int &width, int64_t &src_row,
                                           const uint32_t *&words, int &stride)
{
    if (p >= a.rows) return false;
    int bi = -1;
    for (int u = 0; u < a.nb; ++u)
        if (p >= a.group_info[u] && p < a.group_info[u + 1]) bi = u;
    if (bi < 0) return false;       // beyond the placed rows (a width outside the bit set was skipped)
    width = a.bmin + bi;
    stride = (int)skim_row_stride_words(a.cols, width);
    words = a.packed + a.group_info[a.nb + 1 + bi] + (p - a.group_info[bi]) * (int64_t)stride;
    src_row = a.row_order[p];
    if (!SKIM_IDX(src_row, a.rows, nullptr)) return false;
    return true;
}

// Where entry j of the per-column vector sits in shared memory: inside each block of 256 entries the
// first quads of all 32 lanes come first, then the second quads, so that a lane's 8 entries are two
// 16-byte loads that are contiguous across the warp.
__device__ __forceinline__ int vec_slot(int j)
{
    const int in = j & (STEP - 1), lane = in >> 3, u = in & 7;
    return (j & ~(STEP - 1)) + (u >> 2) * 128 + lane * 4 + (u & 3);
}

constexpr int AHEAD = 4;            // steps whose words are fetched together; two such batches are in flight

// The 8 codes of this lane in a step of B-bit codes, cut out of the step's 8B words (lane l < 8B holds
// word l in `w`), as one word (code u in bits [u*B, (u+1)*B)).
template <int B>
__device__ __forceinline__ uint32_t lane_codes(uint32_t w, int lane)
{
    const int bit = 8 * B * lane;
    const uint32_t lo = __shfl_sync(0xffffffffu, w, bit >> 5);
    const uint32_t hi = __shfl_sync(0xffffffffu, w, (bit >> 5) + 1);
    const uint32_t v = __funnelshift_r(lo, hi, bit & 31);
    return B == 4 ? v : (v & ((1u << (8 * B)) - 1u));
}

template <int B, bool MATVEC>
__device__ __forceinline__ void unpack_row(const UnpackArgs &a, const float *vec, float *book, const uint32_t *words,
                                           int stride, int64_t src_row, int lane)
{
    // the row's codebook, as binary32, in the warp's 16 words of shared memory
    if (lane < 16) book[lane] = lane < a.kmax ? __half2float(__ushort_as_half(a.lut[src_row * a.kmax + lane])) : 0.0f;
    __syncwarp();
    const int steps = (a.cols + STEP - 1) / STEP;
    float acc = 0.0f;
    // the words of the next AHEAD steps are requested before the current ones are worked on
    uint32_t wv[AHEAD], wn[AHEAD];
#pragma unroll
    for (int q = 0; q < AHEAD; ++q) {
        const int w0 = q * 8 * B + lane;                       // lanes 0 .. 8B-1 fetch a step's words
        wv[q] = (lane < 8 * B && w0 < stride) ? __ldg(words + w0) : 0u;
    }
    for (int t0 = 0; t0 < steps; t0 += AHEAD) {
#pragma unroll
        for (int q = 0; q < AHEAD; ++q) {
            const int w0 = (t0 + AHEAD + q) * 8 * B + lane;
            wn[q] = (lane < 8 * B && w0 < stride) ? __ldg(words + w0) : 0u;
        }
#pragma unroll
        for (int q = 0; q < AHEAD; ++q) {
            const int t = t0 + q;
            if (t >= steps) break;
            const uint32_t codes = lane_codes<B>(wv[q], lane);
            const int j0 = t * STEP + lane * 8;
            // the step's 256 vector entries are stored as two runs of quads (see vec_slot): both loads are conflict-free;
            // a dequantiser without a scaling vector has nothing to multiply by and skips them
            const bool use_vec = MATVEC || a.s != nullptr;
            float4 va = make_float4(1.f, 1.f, 1.f, 1.f), vb = va;
            if (use_vec) {
                va = *reinterpret_cast<const float4 *>(vec + t * STEP + lane * 4);
                vb = *reinterpret_cast<const float4 *>(vec + t * STEP + 128 + lane * 4);
            }
            const float v[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
            float r[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float e = book[(codes >> (u * B)) & ((1u << B) - 1u)];
                if (MATVEC) acc = fmaf(e, v[u], acc);
                else r[u] = use_vec ? __fmul_rn(e, v[u]) : e;
            }
            if (!MATVEC) {
                uint16_t *dst = a.out + src_row * a.ld + j0;
                if (a.out_vec && j0 + 8 <= a.cols) {
                    uint32_t h[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        h[u] = (uint32_t)__half_as_ushort(__float2half_rn(r[2 * u])) |
                               ((uint32_t)__half_as_ushort(__float2half_rn(r[2 * u + 1])) << 16);
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(h[0], h[1], h[2], h[3]);
                } else {
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (j0 + u < a.cols) dst[u] = __half_as_ushort(__float2half_rn(r[u]));
                }
            }
        }
#pragma unroll
        for (int q = 0; q < AHEAD; ++q) wv[q] = wn[q];
    }
    if (MATVEC) {
#pragma unroll
        for (int off = 16; off; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) a.y[src_row] = acc;
    }
}

template <bool MATVEC>
__global__ void __launch_bounds__(UT) skim_unpack_kernel(UnpackArgs a)
{
    extern __shared__ __align__(16) float vec[];          // [cols rounded up to STEP], zero beyond cols
    __shared__ float books[UW][16];
    const int padded = (MATVEC || a.s) ? (a.cols + STEP - 1) / STEP * STEP : 0;
    for (int j = threadIdx.x; j < padded; j += UT) {
        float v = 0.0f;
        if (j < a.cols) {
            v = a.s ? a.s[j] : 1.0f;
            if (MATVEC) {
                const float xj = __half2float(__ushort_as_half(a.x[j]));
                v = a.s ? __fmul_rn(xj, v) : xj;
            }
        }
        vec[vec_slot(j)] = v;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // rows are dealt round-robin to the blocks, so that every SM gets the same number (within one)
    for (int64_t p = blockIdx.x + (int64_t)gridDim.x * warp; p < a.rows; p += (int64_t)gridDim.x * UW) {
        int width = 0, stride = 0;
        int64_t src_row = 0;
        const uint32_t *words = nullptr;
        if (!locate_row(a, p, width, src_row, words, stride)) continue;
        __syncwarp();
        switch (width) {
        case 1: unpack_row<1, MATVEC>(a, vec, books[warp], words, stride, src_row, lane); break;
        case 2: unpack_row<2, MATVEC>(a, vec, books[warp], words, stride, src_row, lane); break;
        case 3: unpack_row<3, MATVEC>(a, vec, books[warp], words, stride, src_row, lane); break;
        default: unpack_row<4, MATVEC>(a, vec, books[warp], words, stride, src_row, lane); break;
        }
    }
}

template <bool MATVEC>
int launch_unpack(skim_ctx *ctx, const UnpackArgs &a)
{
    const size_t smem = (size_t)((a.cols + STEP - 1) / STEP * STEP) * sizeof(float);
    if (smem > (size_t)ctx->max_smem_optin) return SKIM_ERR_SHAPE;
    // set on every launch: a host-side call of microseconds, and no state shared between contexts
    SKIM_CUDA_OK(cudaFuncSetAttribute(skim_unpack_kernel<MATVEC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const unsigned blocks = (unsigned)(a.rows < ctx->sm_count ? a.rows : ctx->sm_count);   // one block per SM, rows dealt round-robin
    skim_unpack_kernel<MATVEC><<<blocks, UT, smem, ctx->stream>>>(a);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}

}  // namespace

int skim_launch_dequantize(skim_ctx *ctx, const uint32_t *packed, const int32_t *row_order, const int64_t *group_info,
                           const uint16_t *lut, const float *s, int64_t rows, int64_t cols, const SkimBits &bs,
                           uint16_t *out, int64_t ld_out)
{
    if (rows == 0) return SKIM_OK;
    UnpackArgs a;
    a.packed = packed; a.row_order = row_order; a.group_info = (const long long *)group_info; a.lut = lut;
    a.s = s; a.x = nullptr; a.rows = rows; a.cols = (int)cols; a.nb = bs.n_bits; a.bmin = bs.b_min; a.kmax = 1 << bs.b_max;
    a.out = out; a.ld = ld_out; a.y = nullptr;
    a.out_vec = ((reinterpret_cast<uintptr_t>(out) & 15u) == 0 && (ld_out % 8) == 0) ? 1 : 0;
    return launch_unpack<false>(ctx, a);
}

int skim_launch_matvec(skim_ctx *ctx, const uint32_t *packed, const int32_t *row_order, const int64_t *group_info,
                       const uint16_t *lut, const float *s, const uint16_t *x, int64_t rows, int64_t cols,
                       const SkimBits &bs, float *y)
{
    if (rows == 0) return SKIM_OK;
    UnpackArgs a;
    a.packed = packed; a.row_order = row_order; a.group_info = (const long long *)group_info; a.lut = lut;
    a.s = s; a.x = x; a.rows = rows; a.cols = (int)cols; a.nb = bs.n_bits; a.bmin = bs.b_min; a.kmax = 1 << bs.b_max;
    a.out = nullptr; a.ld = 0; a.out_vec = 0; a.y = y;
    return launch_unpack<true>(ctx, a);
}
