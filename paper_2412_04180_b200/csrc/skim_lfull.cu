// L-full error of every row (SKIM Section 3.4: the layer-wise objective written per row,
// err_i = (w_i - wq_i) X X^T (w_i - wq_i)^T; Section 4.2 and Algorithm 3 fill the error table with it; the
// paper's scaling vector enters through wq = replace(c, l) * alpha, Section 4.3).
//
//   skim_residual_kernel      D = binary16((float(w) - c[label] * alpha) * 2^e): one block per row, labels by the
//                             same midpoint rule as the packer.  Streaming: 2 B in, 2 B out per element.
//   skim_lfull_gemm_kernel    Y = D H (H = X X^T, symmetric, binary16) on the tensor cores and, fused into the
//                             epilogue, the row-wise dot  sum_n Y_in D_in  of every output tile, so Y never
//                             leaves the SM.  This is the one dense contraction of the method.
//   skim_lfull_reduce_kernel  adds the per-tile partial sums of a row in a fixed order, divides 4^e out.
//
// GEMM kernel: persistent, one CTA per SM, tile 128 x 256 x 64, tcgen05.mma (kind::f16, binary32 accumulators
// in tensor memory, two accumulator stages of 256 columns), operands brought in by TMA
// (cp.async.bulk.tensor, 128-byte swizzle) through a 4-stage shared-memory ring.  Warp 0 issues the TMA loads,
// warp 1 allocates tensor memory and issues the MMAs, warps 2-5 read the accumulators back (tcgen05.ld) and do
// the dot product with the matching D tile.  No cluster launch and no multicast: every CTA fetches its own tiles.
// Every wait on an mbarrier is bounded: after WAIT_LIMIT_CYCLES the waiting role raises the block's abort flag,
// sets SKIM_STATUS_TIMEOUT, and all roles leave their loops; tensor memory is freed on every path.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "skim_internal.cuh"

namespace {

// ---------------------------------------------------------------- residual

constexpr int RES_T = 256;

struct ResidualArgs {
    const uint16_t *W;
    const float *rscale;     // 1 / alpha (installed scale), or nullptr
    const float *s;          // alpha itself, or nullptr
    const float *centroids;
    const uint8_t *row_bits; // nullptr: every row at `width`
    int width;
    int64_t ld, ldd;
    int cols;
    int nb, bmin, sumk;
    int exp2;
    int vec;                 // rows of W, D (and of the scale vectors) allow 128-bit accesses
    uint16_t *D;
    unsigned long long *status;
};

__global__ void __launch_bounds__(RES_T) skim_residual_kernel(ResidualArgs a)
{
    __shared__ float tf[16];
    __shared__ float cs[16];
    const int tid = threadIdx.x;
    const int64_t row = blockIdx.x;
    const int b = a.row_bits ? (int)a.row_bits[row] : a.width;
    const int bi = b - a.bmin;
    if (bi < 0 || bi >= a.nb) {
        if (tid == 0) atomicOr(a.status, (unsigned long long)SKIM_STATUS_BAD_BITS);
        return;
    }
    const int k = 1 << b;
    const int off = (1 << a.bmin) * ((1 << bi) - 1);
    const float *c = a.centroids + row * a.sumk + off;
    if (tid < 16) {
        const float cj = c[min(tid, k - 1)];
        cs[tid] = cj;
        float t = __int_as_float(0x7f800000);
        if (tid < k - 1) {
            t = __double2float_rd(0.5 * ((double)cj + (double)c[tid + 1]));
            if (t == 0.0f) t = 0.0f;
        }
        tf[tid] = t;
    }
    __syncthreads();
    const uint16_t *Wr = a.W + row * a.ld;
    uint16_t *Dr = a.D + row * a.ldd;
    const float scale = __int_as_float((127 + a.exp2) << 23);       // 2^exp2, exact
    if (a.vec) {
        // eight elements per thread and step: one 128-bit load of W, one 128-bit store of D
        for (int e0 = tid * 8; e0 < a.cols; e0 += RES_T * 8) {
            const uint4 wv = __ldcs(reinterpret_cast<const uint4 *>(Wr + e0));
            const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
            float rs[8], sv[8];
            if (a.rscale) {
                const float4 r0 = *reinterpret_cast<const float4 *>(a.rscale + e0), r1 = *reinterpret_cast<const float4 *>(a.rscale + e0 + 4);
                rs[0] = r0.x; rs[1] = r0.y; rs[2] = r0.z; rs[3] = r0.w; rs[4] = r1.x; rs[5] = r1.y; rs[6] = r1.z; rs[7] = r1.w;
            }
            if (a.s) {
                const float4 s0 = *reinterpret_cast<const float4 *>(a.s + e0), s1 = *reinterpret_cast<const float4 *>(a.s + e0 + 4);
                sv[0] = s0.x; sv[1] = s0.y; sv[2] = s0.z; sv[3] = s0.w; sv[4] = s1.x; sv[5] = s1.y; sv[6] = s1.z; sv[7] = s1.w;
            }
            uint32_t out[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float w = __half2float(__ushort_as_half((uint16_t)((u & 1) ? (ww[u >> 1] >> 16) : (ww[u >> 1] & 0xffffu))));
                float x = w;
                if (a.rscale) x = __fmul_rn(w, rs[u]);
                int code = (x > tf[7]) ? 8 : 0;
                code += (x > tf[code + 3]) ? 4 : 0;
                code += (x > tf[code + 1]) ? 2 : 0;
                code += (x > tf[code]) ? 1 : 0;
                float q = cs[code];
                if (a.s) q = __fmul_rn(q, sv[u]);
                const uint32_t h = __half_as_ushort(__float2half_rn(__fmul_rn(__fsub_rn(w, q), scale)));
                out[u >> 1] |= h << (16 * (u & 1));
            }
            __stcs(reinterpret_cast<uint4 *>(Dr + e0), make_uint4(out[0], out[1], out[2], out[3]));
        }
        return;
    }
    for (int e = tid; e < a.cols; e += RES_T) {
        const float w = __half2float(__ushort_as_half(Wr[e]));
        float x = w;
        if (a.rscale) x = __fmul_rn(w, a.rscale[e]);
        int code = (x > tf[7]) ? 8 : 0;
        code += (x > tf[code + 3]) ? 4 : 0;
        code += (x > tf[code + 1]) ? 2 : 0;
        code += (x > tf[code]) ? 1 : 0;
        float q = cs[code];
        if (a.s) q = __fmul_rn(q, a.s[e]);
        const float r = __fsub_rn(w, q);
        Dr[e] = __half_as_ushort(__float2half_rn(__fmul_rn(r, scale)));
    }
}

// ---------------------------------------------------------------- GEMM with fused row-wise dot

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int STAGES = 4;
constexpr int UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int GEMM_THREADS = 192;
constexpr int SPLIT_MAX = 8;                    // ranges of K a tile of the last round is cut into, at most
constexpr int TMEM_COLS = 512;                  // two accumulator stages of BN binary32 columns
constexpr long long WAIT_LIMIT_CYCLES = 400000000ll;   // about 0.2 s; a whole launch takes milliseconds
constexpr size_t GEMM_SMEM = (size_t)STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

struct GemmSync {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    int abort;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(smem_u32(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}
// Bounded wait.  False when the block is aborting (this wait ran out, or another role's did).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
            *abort_flag = 1;
            return false;
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
                     smem_u32(dst)),
                 "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
                 : "memory");
}

// Shared-memory operand descriptor: K-major tile whose rows are 64 binary16 = 128 bytes, 128-byte swizzle,
// 8-row groups 1024 bytes apart (the layout TMA writes with CU_TENSOR_MAP_SWIZZLE_128B); tiles are 1024-byte
// aligned, and a step of UMMA_K elements along K inside the swizzle row is a plain 32-byte address offset.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);          // start address
    d |= (uint64_t)1 << 16;                                // leading byte offset (unused for this layout)
    d |= (uint64_t)(1024 >> 4) << 32;                      // stride byte offset: 8 rows x 128 bytes
    d |= (uint64_t)1 << 46;                                // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                                // 128-byte swizzle
    return d;
}

// Instruction descriptor of kind::f16: D binary32, A and B binary16, both K-major, M = 128, N = 256.
constexpr uint32_t IDESC = (1u << 4) | (0u << 7) | (0u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
                 "l"(adesc), "l"(bdesc), "r"(IDESC), "r"(accumulate)
                 : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive binary32 columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t *v)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct GemmArgs {
    const uint16_t *D;       // [rows][ldd] binary16 (also operand A, through its tensor map)
    int64_t ldd;
    int rows, cols;
    int mt, nt;              // tiles along rows and along columns
    int full_tiles, split;   // tiles [full_tiles, mt * nt) are cut into `split` ranges of K (see unit_of)
    float *partial;          // [mt * BM][split][nt]
    float *Y;                // optional [rows][ldy]: the product D H itself (the scaling-vector update needs it)
    int64_t ldy;
    unsigned long long *status;
};

// Work units.  Tiles are taken round-robin by the persistent CTAs; the tiles of the last, partly filled round
// would leave most SMs idle for a whole tile time, so each of them is cut into `split` ranges of K that run
// side by side.  The fused row-wise dot is linear in the accumulator, so a range simply leaves one more partial
// dot per row (column `slice` of the partial array); the product Y itself is only written by unsplit launches.
struct GemmUnit {
    int tile, slice, kb0, kb1;
};
__device__ __forceinline__ GemmUnit unit_of(const GemmArgs &a, int u, int nkb)
{
    GemmUnit w;
    if (u < a.full_tiles) {
        w.tile = u; w.slice = 0; w.kb0 = 0; w.kb1 = nkb;
    } else {
        const int r = u - a.full_tiles;
        w.tile = a.full_tiles + r / a.split;
        w.slice = r % a.split;
        w.kb0 = (int)((long long)nkb * w.slice / a.split);
        w.kb1 = (int)((long long)nkb * (w.slice + 1) / a.split);
    }
    return w;
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
skim_lfull_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, GemmArgs a)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *tiles = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    GemmSync &sy = *reinterpret_cast<GemmSync *>(tiles + (size_t)STAGES * STAGE_BYTES);
    volatile int *abort_flag = &sy.abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = (a.cols + BK - 1) / BK;
    const int ntiles = a.mt * a.nt;
    const int nunits = a.full_tiles + (ntiles - a.full_tiles) * a.split;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&sy.full[s], 1); mbar_init(&sy.empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&sy.tmem_full[s], 1); mbar_init(&sy.tmem_empty[s], 4); }
        sy.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sy.tmem_base)), "r"(TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sy.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (one lane)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < nunits && ok; u += gridDim.x) {
                const GemmUnit w = unit_of(a, u, nkb);
                const int m0 = (w.tile % a.mt) * BM, n0 = (w.tile / a.mt) * BN;
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    if (!(ok = mbar_wait(&sy.empty[stage], phase ^ 1u, abort_flag))) break;
                    unsigned char *sa = tiles + (size_t)stage * STAGE_BYTES;
                    mbar_expect_tx(&sy.full[stage], STAGE_BYTES);
                    tma_load_2d(sa, &map_a, &sy.full[stage], kb * BK, m0);
                    tma_load_2d(sa + A_BYTES, &map_b, &sy.full[stage], kb * BK, n0);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one lane)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (int u = blockIdx.x; u < nunits && ok; u += gridDim.x, ++it) {
                const GemmUnit w = unit_of(a, u, nkb);
                const int as = it & 1;
                if (!(ok = mbar_wait(&sy.tmem_empty[as], (((uint32_t)it >> 1) & 1u) ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(as * BN);
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    if (!(ok = mbar_wait(&sy.full[stage], phase, abort_flag))) break;
                    tc_fence_after();
                    const uint32_t sa = smem_u32(tiles + (size_t)stage * STAGE_BYTES), sb = sa + A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_f16(tmem_d, umma_desc(sa + k * UMMA_K * 2), umma_desc(sb + k * UMMA_K * 2), (kb > w.kb0 || k) ? 1u : 0u);
                    umma_commit(&sy.empty[stage]);           // the stage is free once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(&sy.tmem_full[as]);      // the accumulator is complete once all MMAs are
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: 4 warps, one row per thread
        const int q = warp & 3;                               // the tensor-memory lane quarter this warp may read
        bool ok = true;
        int it = 0;
        for (int u = blockIdx.x; u < nunits && ok; u += gridDim.x, ++it) {
            const GemmUnit w = unit_of(a, u, nkb);
            const int as = it & 1;
            const int mb = w.tile % a.mt, nb = w.tile / a.mt;
            const int row = mb * BM + q * 32 + lane;
            const int n0 = nb * BN;
            const uint16_t *drow = a.D + (int64_t)min(row, a.rows - 1) * a.ldd;
            ok = mbar_wait(&sy.tmem_full[as], ((uint32_t)it >> 1) & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            float acc = 0.0f;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                const int col = n0 + c * 32;
                uint4 dv[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    dv[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (col + u * 8 + 8 <= a.cols) dv[u] = __ldg(reinterpret_cast<const uint4 *>(drow + col + u * 8));
                }
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN + c * 32), v);
                if (a.Y && row < a.rows) {
                    float *yrow = a.Y + (int64_t)row * a.ldy + col;
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (col + u * 4 + 4 <= a.cols)
                            *reinterpret_cast<uint4 *>(yrow + u * 4) = make_uint4(v[u * 4], v[u * 4 + 1], v[u * 4 + 2], v[u * 4 + 3]);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t w4[4] = {dv[u].x, dv[u].y, dv[u].z, dv[u].w};
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w4[h]));
                        acc = fmaf(__uint_as_float(v[u * 8 + 2 * h]), f.x, acc);
                        acc = fmaf(__uint_as_float(v[u * 8 + 2 * h + 1]), f.y, acc);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sy.tmem_empty[as]);
            if (row < a.rows) a.partial[((int64_t)row * a.split + w.slice) * a.nt + nb] = acc;
        }
    }
    // ---------------------------------------------------------------- teardown (every path comes here)
    tc_fence_before();
    __syncthreads();
    if (sy.abort) {
        // a wait ran out: give the bulk copies that may still be in flight time to land before the block's
        // shared memory is released (about a millisecond), and report
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        if (threadIdx.x == 0) atomicOr(a.status, (unsigned long long)SKIM_STATUS_TIMEOUT);
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS));
    }
}

// Adds a row's partial dots in a fixed order: slice 0 of every column tile, then the further slices of the tiles
// that were cut along K (only those entries were written).
__global__ void skim_lfull_reduce_kernel(const float *__restrict__ partial, int rows, int mt, int nt, int full_tiles, int split,
                                         int exp2, float *__restrict__ err, int64_t err_stride, double *__restrict__ err64)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    const int mb = i / BM;
    double s = 0.0;
    for (int t = 0; t < nt; ++t) s += (double)partial[((int64_t)i * split) * nt + t];
    for (int sl = 1; sl < split; ++sl)
        for (int t = 0; t < nt; ++t)
            if (t * mt + mb >= full_tiles) s += (double)partial[((int64_t)i * split + sl) * nt + t];
    if (err) err[(int64_t)i * err_stride] = (float)ldexp(s, -2 * exp2);
    if (err64) err64[i] = ldexp(s, -2 * exp2);
}

int encode_map(CUtensorMap *map, const uint16_t *base, int64_t rows, int64_t cols, int64_t ld, int box_rows)
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn)
        return SKIM_ERR_CUDA;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn)(
        map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<uint16_t *>(base), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SKIM_OK : SKIM_ERR_CUDA;
}

}  // namespace

int skim_launch_residual(skim_ctx *ctx, const uint16_t *W, int64_t rows, int64_t cols, int64_t ld, const float *centroids,
                         const uint8_t *row_bits, int width, const SkimBits &bs, const float *s, int exp2, uint16_t *D,
                         int64_t ldd)
{
    if (rows == 0) return SKIM_OK;
    SkimWorkspace ws = skim_carve(ctx->ws, rows, cols);
    ResidualArgs a;
    a.W = W;
    a.rscale = ctx->scaled ? ws.rscale : nullptr;
    a.s = s;
    a.centroids = centroids;
    a.row_bits = row_bits;
    a.width = width;
    a.ld = ld;
    a.ldd = ldd;
    a.cols = (int)cols;
    a.nb = bs.n_bits;
    a.bmin = bs.b_min;
    a.sumk = bs.sumk;
    a.exp2 = exp2;
    a.vec = ((reinterpret_cast<uintptr_t>(W) & 15u) == 0 && (reinterpret_cast<uintptr_t>(D) & 15u) == 0 && ld % 8 == 0 &&
             ldd % 8 == 0 && cols % 8 == 0 && (!s || (reinterpret_cast<uintptr_t>(s) & 15u) == 0)) ? 1 : 0;
    a.D = D;
    a.status = ws.status;
    skim_residual_kernel<<<(unsigned)rows, RES_T, 0, ctx->stream>>>(a);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}

size_t skim_lfull_scratch_bytes(int64_t rows, int64_t cols)
{
    const int64_t mt = (rows + BM - 1) / BM, nt = (cols + BN - 1) / BN;
    return skim_align256((size_t)(mt * BM) * (size_t)nt * SPLIT_MAX * sizeof(float));
}

int skim_launch_err_lfull(skim_ctx *ctx, const uint16_t *D, int64_t rows, int64_t cols, int64_t ldd, const uint16_t *H,
                          int64_t ldh, int exp2, void *scratch, float *err, int64_t err_stride, float *Y, int64_t ldy,
                          double *err64)
{
    if (rows == 0) return SKIM_OK;
    CUtensorMap map_a, map_b;
    int rc = encode_map(&map_a, D, rows, cols, ldd, BM);
    if (rc) return rc;
    rc = encode_map(&map_b, H, cols, cols, ldh, BN);
    if (rc) return rc;
    GemmArgs a;
    a.D = D;
    a.ldd = ldd;
    a.rows = (int)rows;
    a.cols = (int)cols;
    a.mt = (int)((rows + BM - 1) / BM);
    a.nt = (int)((cols + BN - 1) / BN);
    a.partial = (float *)scratch;
    a.Y = Y;
    a.ldy = ldy;
    a.status = (unsigned long long *)ctx->ws;
    SKIM_CUDA_OK(cudaFuncSetAttribute(skim_lfull_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM_SMEM));
    const int tiles = a.mt * a.nt;
    // the tiles of the last round, if it is not full, are cut along K into as many ranges as fit the SMs
    const int nkb = (int)((cols + BK - 1) / BK);
    const int rest = tiles % ctx->sm_count;
    a.full_tiles = tiles;
    a.split = 1;
    if (!Y && rest > 0) {
        // `rest` tiles in s ranges each take ceil(rest s / SMs) sub-rounds of 1/s tile time: the least, the smaller s on a tie
        int sp = 1;
        double best = 1.0;
        for (int c = 2; c <= SPLIT_MAX && c <= nkb; ++c) {
            const double cost = (double)((rest * c + ctx->sm_count - 1) / ctx->sm_count) / c;
            if (cost < best - 1e-9) { best = cost; sp = c; }
        }
        if (sp > 1) {
            a.full_tiles = tiles - rest;
            a.split = sp;
        }
    }
    const int units = a.full_tiles + (tiles - a.full_tiles) * a.split;
    const unsigned blocks = (unsigned)(units < ctx->sm_count ? units : ctx->sm_count);    // persistent: one CTA per SM
    skim_lfull_gemm_kernel<<<blocks, GEMM_THREADS, GEMM_SMEM, ctx->stream>>>(map_a, map_b, a);
    SKIM_CUDA_OK(cudaGetLastError());
    skim_lfull_reduce_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, ctx->stream>>>(a.partial, (int)rows, a.mt, a.nt, a.full_tiles, a.split, exp2, err,
                                                                                      err_stride, err64);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 2;
    return SKIM_OK;
}
