// Scaling-vector training with the labels held fixed (SKIM Section 4.3, Algorithm 2, inner
// repeat; optimiser settings of Section 5.1).
//
//   loss(alpha) = sum_ij g_ij (W_ij - alpha_j c_{i,l_ij})^2,
//   c_ik        = sum_{j in k} g_ij W_ij / alpha_j  /  sum_{j in k} g_ij   (re-fitted each step)
//
// Per Adam step the matrix is read twice, by two kernels:
//   skim_scale_sums_kernel  one warp per row.  Per cluster k of the row it forms, in binary64,
//       S_k = sum g w / alpha,  A_k = sum g w alpha,  B_k = sum g alpha^2  (sums over the members).
//       With the per-call constants G_k = sum g and D_k = sum g w^2 (the same kernel, run once in
//       its INIT form) these give the centroid c_k = S_k / G_k, the row's loss
//       sum_k D_k - 2 c_k A_k + c_k^2 B_k, and the factor q_k = 2 (A_k - c_k B_k) / G_k through which the
//       re-fitted centroid enters the gradient -- without a second pass over the row.  A lane adds
//       its elements into accumulator slots of its own in shared memory (one per cluster and
//       sum), so no atomics are needed and every sum has a fixed order.
//   skim_scale_grad_kernel  a thread owns four columns and walks a range of rows:
//       d loss / d alpha_j = sum_i  -2 g c (w - alpha_j c) + q g w / alpha_j^2   (c, q of the element's
//       cluster, read from the 512-byte table the first kernel left for the row), accumulated in
//       registers; the row ranges leave partial gradients that the Adam kernel adds in a fixed order.
//   skim_scale_adam_kernel  sums the partials and the rows' losses (deterministic), applies the
//       Adam update to the binary64 master copy of alpha and to its lane-interleaved copy, the
//       one the row-wise kernels read (alpha_il_pos).
#include "skim_internal.cuh"

namespace {

constexpr int KC = 16;      // clusters per row at most (4 bits)
constexpr int SW = 4;       // warps (rows) per block of the sums kernel
constexpr int NSUM = 3;
constexpr int GW = 2;       // elements whose slot updates of the sums kernel go together
constexpr int GT = 256;     // threads of a gradient block
constexpr int GC = 4;       // columns per thread

struct ScaleArgs {
    const uint16_t *W;
    const float *G;
    const uint8_t *labels;
    const double *alpha;
    const double *alpha_il; // alpha in the lane-interleaved order of alpha_il_pos()
    int64_t rows, ld;
    int cols;
    int vec;                // rows of W, G and labels allow the vector loads of both kernels
    double2 *tconst;        // [rows][KC]  (G_k, D_k)
    double2 *tq;            // [rows][KC]  (c_k, q_k)
    double *loss_row;       // [rows]
    double *grad_part;      // [row ranges][cols]
    int rows_per_range;
};

// A lane of the row-wise kernels owns eight consecutive columns of every 256 and reads their alphas two at a
// time.  From the plain array those reads are 64 bytes apart across the lanes (sixteen 128-byte wavefronts of the
// L1 data path for 512 useful bytes, and that path is what bounds the sums kernel); from this order -- the u-th
// pair of lane L at 64 u + 2 L of its block of 256 -- a warp's read is one contiguous 512 bytes.
__host__ __device__ __forceinline__ int alpha_il_pos(int j)
{
    const int r = j & 255;
    return (j & ~255) + 64 * ((r >> 1) & 3) + 2 * (r >> 3) + (r & 1);
}

// 1 / a for a positive, normal binary64 a (the scale vector is checked to be that): the hardware's approximate
// reciprocal (about 23 bits) and two Newton steps, within one unit in the last place.  Five instructions where the
// correctly rounded division-free reciprocal takes about twelve; the sums kernel needs one per element.
__device__ __forceinline__ double rcp_pos(double a)
{
    double r;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(a));
    r = fma(r, fma(-a, r, 1.0), r);
    return fma(r, fma(-a, r, 1.0), r);
}

// Eight consecutive elements of a row starting at e0 (a multiple of 8), as loaded; entries at or
// beyond cols come back with zero importance, label 0 and alpha 1.
struct Raw8 {
    uint4 w;            // 8 binary16 weights
    float4 ga, gb;      // 8 importances
    uint2 l;            // 8 labels
    double2 al[4];      // 8 alphas
};

template <bool VEC>
__device__ __forceinline__ void load8(const ScaleArgs &a, int64_t row, int e0, Raw8 &r)
{
    const uint16_t *Wr = a.W + row * a.ld;
    const float *Gr = a.G + row * a.ld;
    const uint8_t *Lr = a.labels + row * (int64_t)a.cols;
    if (VEC && e0 + 8 <= a.cols) {
        // the matrix streams through once per kernel: keep it from evicting alpha
        r.w = __ldcs(reinterpret_cast<const uint4 *>(Wr + e0));
        r.ga = __ldcs(reinterpret_cast<const float4 *>(Gr + e0));
        r.gb = __ldcs(reinterpret_cast<const float4 *>(Gr + e0 + 4));
        r.l = __ldcs(reinterpret_cast<const uint2 *>(Lr + e0));
#pragma unroll
        for (int u = 0; u < 4; ++u) r.al[u] = __ldg(reinterpret_cast<const double2 *>(a.alpha_il + alpha_il_pos(e0 + 2 * u)));
    } else {
        uint32_t ww[4] = {0u, 0u, 0u, 0u}, ll[2] = {0u, 0u};
        float gg[8];
        double aa[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const bool in = e0 + u < a.cols;
            ww[u >> 1] |= (in ? (uint32_t)Wr[e0 + u] : 0u) << (16 * (u & 1));
            ll[u >> 2] |= (in ? (uint32_t)(Lr[e0 + u] & (KC - 1)) : 0u) << (8 * (u & 3));
            gg[u] = in ? Gr[e0 + u] : 0.0f;
            aa[u] = in ? a.alpha[e0 + u] : 1.0;
        }
        r.w = make_uint4(ww[0], ww[1], ww[2], ww[3]);
        r.ga = make_float4(gg[0], gg[1], gg[2], gg[3]);
        r.gb = make_float4(gg[4], gg[5], gg[6], gg[7]);
        r.l = make_uint2(ll[0], ll[1]);
#pragma unroll
        for (int u = 0; u < 4; ++u) r.al[u] = make_double2(aa[2 * u], aa[2 * u + 1]);
    }
}

// Adds W (2 or 4) elements' terms to the lane's accumulator slots.  The slots of a sum are read together and the
// additions then run in element order in registers, an element whose cluster matches an earlier one of the
// group continuing from that one's result: the same sums in the same order as one read-modify-write after
// another, without the round trips through shared memory in a row.
template <int NS, int W>
__device__ __forceinline__ void add_group(double *slot, const int (&l)[8], const double (&cs)[NS][8], int u0)
{
    double v[NS][W];
#pragma unroll
    for (int s = 0; s < NS; ++s)
#pragma unroll
        for (int u = 0; u < W; ++u) v[s][u] = slot[(s * KC + l[u0 + u]) * 32];
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        double n[W];
#pragma unroll
        for (int u = 0; u < W; ++u) {
            double base = v[s][u];
#pragma unroll
            for (int t = 0; t < u; ++t)
                if (l[u0 + t] == l[u0 + u]) base = n[t];          // the latest earlier element of the cluster wins
            n[u] = base + cs[s][u0 + u];
        }
        // in element order: where clusters repeat, the last store holds the full sum
#pragma unroll
        for (int u = 0; u < W; ++u) slot[(s * KC + l[u0 + u]) * 32] = n[u];
    }
}

// INIT: the per-call constants (G_k, D_k) of every row.  Otherwise: (c_k, q_k) and the row's loss.
template <bool INIT, bool VEC>
__global__ void __launch_bounds__(SW * 32) skim_scale_sums_kernel(ScaleArgs a)
{
    extern __shared__ __align__(16) double slots_all[];       // [SW][NSUM * KC][32]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * SW + warp;
    if (row >= a.rows) return;
    double *slot = slots_all + (size_t)warp * (NSUM * KC * 32) + lane;   // entry (s, k) at slot[(s * KC + k) * 32]
#pragma unroll
    for (int q = 0; q < NSUM * KC; ++q) slot[q * 32] = 0.0;
    // the loads of the next step are issued before the current one is worked on
    Raw8 cur, nxt;
    if (lane * 8 < a.cols) load8<VEC>(a, row, lane * 8, cur);
    for (int e0 = lane * 8; e0 < a.cols; e0 += 256) {
        if (e0 + 256 < a.cols) load8<VEC>(a, row, e0 + 256, nxt);
        const uint32_t ww[4] = {cur.w.x, cur.w.y, cur.w.z, cur.w.w};
        const float g[8] = {cur.ga.x, cur.ga.y, cur.ga.z, cur.ga.w, cur.gb.x, cur.gb.y, cur.gb.z, cur.gb.w};
        const double al[8] = {cur.al[0].x, cur.al[0].y, cur.al[1].x, cur.al[1].y, cur.al[2].x, cur.al[2].y, cur.al[3].x, cur.al[3].y};
        int l[8];
        double cs[INIT ? 2 : NSUM][8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float wf = __half2float(__ushort_as_half((uint16_t)((u & 1) ? (ww[u >> 1] >> 16) : (ww[u >> 1] & 0xffffu))));
            l[u] = (int)(((u < 4 ? cur.l.x : cur.l.y) >> (8 * (u & 3))) & (KC - 1));
            const double gd = (double)g[u], wd = (double)wf;
            const double gw = gd * wd;
            if (INIT) {
                cs[0][u] = gd;
                cs[1][u] = gw * wd;
            } else {
                cs[0][u] = gw * rcp_pos(al[u]);
                cs[1][u] = gw * al[u];
                cs[2][u] = gd * al[u] * al[u];
            }
        }
#pragma unroll
        for (int u0 = 0; u0 < 8; u0 += GW) add_group<INIT ? 2 : NSUM, GW>(slot, l, cs, u0);
        cur = nxt;
    }
    __syncwarp();
    // lane L adds up entry L (and L + 32) over the 32 lanes' slots, starting at its own (no bank conflicts)
    const double *base = slots_all + (size_t)warp * (NSUM * KC * 32);
    double v0 = 0.0, v1 = 0.0;
    for (int t = 0; t < 32; ++t) {
        const int src = (t + lane) & 31;
        v0 += base[lane * 32 + src];
        if (lane < NSUM * KC - 32) v1 += base[(lane + 32) * 32 + src];
    }
    // sums 0 and 1 of cluster k sit in lanes k and 16 + k (v0), sum 2 in lane k (v1)
    const double s0 = v0, s1 = __shfl_sync(0xffffffffu, v0, (lane & 15) + 16), s2 = v1;
    double loss_k = 0.0;
    if (lane < KC) {
        if (INIT) {
            a.tconst[row * KC + lane] = make_double2(s0, s1);
        } else {
            const double2 gdk = a.tconst[row * KC + lane];
            double c = 0.0, q = 0.0;
            if (gdk.x > 0.0) {
                c = s0 / gdk.x;
                q = 2.0 * (s1 - c * s2) / gdk.x;
                loss_k = gdk.y - 2.0 * c * s1 + c * c * s2;
            }
            a.tq[row * KC + lane] = make_double2(c, q);
        }
    }
    if (!INIT) {
#pragma unroll
        for (int off = 8; off; off >>= 1) loss_k += __shfl_down_sync(0xffffffffu, loss_k, off);
        if (lane == 0) a.loss_row[row] = loss_k;
    }
}

// The W, G and label entries of one thread's four columns in RB consecutive rows, as loaded.
template <int RB>
struct GradRows {
    uint2 wv[RB];
    float4 gv[RB];
    uint32_t lv[RB];
};

template <bool VEC, int RB>
__device__ __forceinline__ void grad_load(const ScaleArgs &a, int64_t rb, int64_t r1, int j0, bool full, GradRows<RB> &r)
{
#pragma unroll
    for (int q = 0; q < RB; ++q) {
        const int64_t row = rb + q;
        r.wv[q] = make_uint2(0u, 0u); r.gv[q] = make_float4(0.f, 0.f, 0.f, 0.f); r.lv[q] = 0u;
        if (row < r1 && j0 < a.cols) {
            const uint16_t *Wr = a.W + row * a.ld + j0;
            const float *Gr = a.G + row * a.ld + j0;
            const uint8_t *Lr = a.labels + row * (int64_t)a.cols + j0;
            if (full) {
                r.wv[q] = __ldcs(reinterpret_cast<const uint2 *>(Wr));
                r.gv[q] = __ldcs(reinterpret_cast<const float4 *>(Gr));
                r.lv[q] = __ldcs(reinterpret_cast<const uint32_t *>(Lr));
            } else {
                uint32_t ww[2] = {0u, 0u};
                float gg[GC];
#pragma unroll
                for (int u = 0; u < GC; ++u) {
                    const bool in = j0 + u < a.cols;
                    ww[u >> 1] |= (in ? (uint32_t)Wr[u] : 0u) << (16 * (u & 1));
                    r.lv[q] |= (in ? (uint32_t)(Lr[u] & (KC - 1)) : 0u) << (8 * u);
                    gg[u] = in ? Gr[u] : 0.0f;
                }
                r.wv[q] = make_uint2(ww[0], ww[1]);
                r.gv[q] = make_float4(gg[0], gg[1], gg[2], gg[3]);
            }
        }
    }
}

template <bool VEC>
__global__ void __launch_bounds__(GT) skim_scale_grad_kernel(ScaleArgs a)
{
    // Rows go by in batches of RB.  While a batch is worked on, the next batch's loads are in flight and its
    // (c_k, q_k) tables wait in a register of the first RB * KC threads; the tables alternate between two buffers,
    // so one barrier per batch is enough.
    constexpr int RB = 4;
    __shared__ double2 tq_s[2][RB * KC];
    const int j0 = (blockIdx.x * GT + threadIdx.x) * GC;
    const int64_t r0 = (int64_t)blockIdx.y * a.rows_per_range;
    const int64_t r1 = min(a.rows, r0 + a.rows_per_range);
    double al[GC], rr[GC], acc[GC];
#pragma unroll
    for (int u = 0; u < GC; ++u) {
        al[u] = j0 + u < a.cols ? a.alpha[j0 + u] : 1.0;
        const double r = __drcp_rn(al[u]);
        rr[u] = r * r;
        acc[u] = 0.0;
    }
    const bool full = VEC && j0 + GC <= a.cols;
    const bool tq_thread = threadIdx.x < RB * KC;
    GradRows<RB> cur, nxt;
    grad_load<VEC, RB>(a, r0, r1, j0, full, cur);
    if (tq_thread && r0 + threadIdx.x / KC < r1) tq_s[0][threadIdx.x] = a.tq[r0 * KC + threadIdx.x];
    int buf = 0;
    for (int64_t rb = r0; rb < r1; rb += RB, buf ^= 1) {
        const int64_t rn = rb + RB;
        double2 tnext = make_double2(0.0, 0.0);
        if (rn < r1) {
            grad_load<VEC, RB>(a, rn, r1, j0, full, nxt);
            if (tq_thread && rn + threadIdx.x / KC < r1) tnext = a.tq[rn * KC + threadIdx.x];
        }
        __syncthreads();                        // this batch's tables are in place; the other buffer is no longer read
#pragma unroll
        for (int q = 0; q < RB; ++q) {
            const int64_t row = rb + q;
            if (row >= r1) break;
            const double2 *tq = tq_s[buf] + q * KC;
            const uint32_t ww[2] = {cur.wv[q].x, cur.wv[q].y};
            const float g[GC] = {cur.gv[q].x, cur.gv[q].y, cur.gv[q].z, cur.gv[q].w};
#pragma unroll
            for (int u = 0; u < GC; ++u) {
                const double2 cq = tq[(cur.lv[q] >> (8 * u)) & (KC - 1)];
                const double gd = (double)g[u];
                const double wd = (double)__half2float(__ushort_as_half((uint16_t)((u & 1) ? (ww[u >> 1] >> 16) : (ww[u >> 1] & 0xffffu))));
                const double res = wd - al[u] * cq.x;
                acc[u] += gd * (cq.y * wd * rr[u] - 2.0 * cq.x * res);
            }
        }
        if (tq_thread) tq_s[buf ^ 1][threadIdx.x] = tnext;
        cur = nxt;
    }
#pragma unroll
    for (int u = 0; u < GC; ++u)
        if (j0 + u < a.cols) a.grad_part[(int64_t)blockIdx.y * a.cols + j0 + u] = acc[u];
}

__global__ void __launch_bounds__(256) skim_scale_adam_kernel(const double *__restrict__ grad_part,
                                                               const double *__restrict__ loss_row, int nranges,
                                                               int64_t rows, int cols, double *alpha, double *alpha_il,
                                                               double *m1, double *m2, double lr, double beta1, double beta2,
                                                               double bc1, double bc2, double eps, double *loss_out)
{
    __shared__ double red[256];
    if (blockIdx.x == gridDim.x - 1) {
        // the last block adds the rows' losses: strided partial sums, then a fixed tree
        double s = 0.0;
        for (int64_t i = threadIdx.x; i < rows; i += 256) s += loss_row[i];
        red[threadIdx.x] = s;
        __syncthreads();
        for (int off = 128; off; off >>= 1) {
            if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
            __syncthreads();
        }
        if (threadIdx.x == 0 && loss_out) *loss_out = red[0];
        return;
    }
    // 32 columns a block; the row ranges' partial gradients are dealt to 8 groups of threads, and the groups' sums
    // are added in a fixed order
    const int c = threadIdx.x & 31, sgrp = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + c;
    double gs = 0.0;
    if (j < cols)
        for (int b = sgrp; b < nranges; b += 8) gs += grad_part[(int64_t)b * cols + j];
    red[threadIdx.x] = gs;
    __syncthreads();
    if (sgrp != 0 || j >= cols) return;
    double g = 0.0;
#pragma unroll
    for (int q = 0; q < 8; ++q) g += red[q * 32 + c];
    const double a1 = beta1 * m1[j] + (1.0 - beta1) * g;
    const double a2 = beta2 * m2[j] + (1.0 - beta2) * g * g;
    m1[j] = a1;
    m2[j] = a2;
    const double an = alpha[j] - lr * (a1 / bc1) / (sqrt(a2 / bc2) + eps);
    alpha[j] = an;
    alpha_il[alpha_il_pos(j)] = an;
}

__global__ void skim_scale_init_kernel(const float *__restrict__ alpha32, int cols, double *alpha, double *alpha_il,
                                       double *m1, double *m2, unsigned long long *status)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= cols) return;
    const float v = alpha32[j];
    if (!(v > 0.0f) || v > 3.0e38f) atomicOr(status, (unsigned long long)SKIM_STATUS_BAD_SCALE);
    alpha[j] = (double)v;
    alpha_il[alpha_il_pos(j)] = (double)v;
    m1[j] = 0.0;
    m2[j] = 0.0;
}

__global__ void skim_scale_finish_kernel(const double *__restrict__ alpha, int cols, float *__restrict__ alpha32)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < cols) alpha32[j] = (float)alpha[j];
}

// ---------------------------------------------------------------- the same update on the L-full loss
//
//   loss(alpha) = sum_i d_i H d_i^T,  d_ij = W_ij - alpha_j c_{i,l_ij},  H = X X^T   (Section 4.3 with the L-full form of
//   Section 3.4).  With Y = D H:  d loss / d alpha_j = sum_i -2 Y_ij c_{i,l} + q_{i,l} g_ij W_ij / alpha_j^2,
//   q_ik = 2 R_ik / G_ik,  R_ik = sum_{j in k} Y_ij alpha_j.
// Per Adam step: skim_scale_lf_residual_kernel (centroids of the step, residual as the binary16 operand of the
// contraction), the tcgen05 GEMM of skim_lfull.cu (Y = D H stored, row-wise dot = the loss), skim_scale_lf_r_kernel
// (R_ik, q_ik), skim_scale_lf_grad_kernel (column sums), and the Adam kernel above.

struct ScaleLfArgs {
    ScaleArgs s;
    uint16_t *D;         // [rows][cols] binary16 residual * 2^exp2
    const float *Y;      // [rows][cols] binary32, D H
    int exp2;
};

// One warp per row: S_k = sum g w / alpha per cluster, c_k = S_k / G_k, then the row of D.
__global__ void __launch_bounds__(SW * 32) skim_scale_lf_residual_kernel(ScaleLfArgs b)
{
    extern __shared__ __align__(16) double slots_all[];       // [SW][KC][32], then [SW][KC] centroids
    const ScaleArgs &a = b.s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * SW + warp;
    if (row >= a.rows) return;
    double *slot = slots_all + (size_t)warp * (KC * 32) + lane;
    double *cs = slots_all + (size_t)SW * (KC * 32) + warp * KC;
#pragma unroll
    for (int q = 0; q < KC; ++q) slot[q * 32] = 0.0;
    Raw8 cur, nxt;
    if (lane * 8 < a.cols) load8<true>(a, row, lane * 8, cur);
    for (int e0 = lane * 8; e0 < a.cols; e0 += 256) {
        if (e0 + 256 < a.cols) load8<true>(a, row, e0 + 256, nxt);
        const uint32_t ww[4] = {cur.w.x, cur.w.y, cur.w.z, cur.w.w};
        const float g[8] = {cur.ga.x, cur.ga.y, cur.ga.z, cur.ga.w, cur.gb.x, cur.gb.y, cur.gb.z, cur.gb.w};
        const double al[8] = {cur.al[0].x, cur.al[0].y, cur.al[1].x, cur.al[1].y, cur.al[2].x, cur.al[2].y, cur.al[3].x, cur.al[3].y};
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float wf = __half2float(__ushort_as_half((uint16_t)((u & 1) ? (ww[u >> 1] >> 16) : (ww[u >> 1] & 0xffffu))));
            const int l = (int)(((u < 4 ? cur.l.x : cur.l.y) >> (8 * (u & 3))) & (KC - 1));
            slot[l * 32] += ((double)g[u] * (double)wf) * rcp_pos(al[u]);
        }
        cur = nxt;
    }
    __syncwarp();
    if (lane < KC) {
        const double *base = slots_all + (size_t)warp * (KC * 32) + lane * 32;
        double v = 0.0;
        for (int t = 0; t < 32; ++t) v += base[(t + lane) & 31];
        const double gk = a.tconst[row * KC + lane].x;
        const double c = gk > 0.0 ? v / gk : 0.0;
        cs[lane] = c;
        a.tq[row * KC + lane] = make_double2(c, 0.0);
    }
    __syncwarp();
    const float scale = __int_as_float((127 + b.exp2) << 23);
    const uint16_t *Wr = a.W + row * a.ld;
    const uint8_t *Lr = a.labels + row * (int64_t)a.cols;
    uint16_t *Dr = b.D + row * (int64_t)a.cols;
    for (int e0 = lane * 8; e0 < a.cols; e0 += 256) {
        const uint4 wv = *reinterpret_cast<const uint4 *>(Wr + e0);
        const uint2 lv = *reinterpret_cast<const uint2 *>(Lr + e0);
        double al[8];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const double2 t = __ldg(reinterpret_cast<const double2 *>(a.alpha_il + alpha_il_pos(e0 + 2 * u)));
            al[2 * u] = t.x;
            al[2 * u + 1] = t.y;
        }
        const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
        uint32_t out[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float wf = __half2float(__ushort_as_half((uint16_t)((u & 1) ? (ww[u >> 1] >> 16) : (ww[u >> 1] & 0xffffu))));
            const int l = (int)(((u < 4 ? lv.x : lv.y) >> (8 * (u & 3))) & (KC - 1));
            const double d = (double)wf - al[u] * cs[l];
            const uint32_t h = __half_as_ushort(__float2half_rn(__fmul_rn((float)d, scale)));
            out[u >> 1] |= h << (16 * (u & 1));
        }
        *reinterpret_cast<uint4 *>(Dr + e0) = make_uint4(out[0], out[1], out[2], out[3]);
    }
}

// One warp per row: R_k = sum_{j in k} Y_ij alpha_j, q_k = 2 R_k / (2^exp2 G_k) into the row's table.
__global__ void __launch_bounds__(SW * 32) skim_scale_lf_r_kernel(ScaleLfArgs b)
{
    extern __shared__ __align__(16) double slots_all[];       // [SW][KC][32]
    const ScaleArgs &a = b.s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * SW + warp;
    if (row >= a.rows) return;
    double *slot = slots_all + (size_t)warp * (KC * 32) + lane;
#pragma unroll
    for (int q = 0; q < KC; ++q) slot[q * 32] = 0.0;
    const float *Yr = b.Y + row * (int64_t)a.cols;
    const uint8_t *Lr = a.labels + row * (int64_t)a.cols;
    for (int e0 = lane * 8; e0 < a.cols; e0 += 256) {
        const float4 ya = __ldcs(reinterpret_cast<const float4 *>(Yr + e0)), yb = __ldcs(reinterpret_cast<const float4 *>(Yr + e0 + 4));
        const uint2 lv = __ldcs(reinterpret_cast<const uint2 *>(Lr + e0));
        const float y[8] = {ya.x, ya.y, ya.z, ya.w, yb.x, yb.y, yb.z, yb.w};
        double al[8];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const double2 t = __ldg(reinterpret_cast<const double2 *>(a.alpha_il + alpha_il_pos(e0 + 2 * u)));
            al[2 * u] = t.x;
            al[2 * u + 1] = t.y;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int l = (int)(((u < 4 ? lv.x : lv.y) >> (8 * (u & 3))) & (KC - 1));
            slot[l * 32] += (double)y[u] * al[u];
        }
    }
    __syncwarp();
    if (lane < KC) {
        const double *base = slots_all + (size_t)warp * (KC * 32) + lane * 32;
        double v = 0.0;
        for (int t = 0; t < 32; ++t) v += base[(t + lane) & 31];
        const double gk = a.tconst[row * KC + lane].x;
        double2 cq = a.tq[row * KC + lane];
        cq.y = gk > 0.0 ? ldexp(2.0 * v, -b.exp2) / gk : 0.0;
        a.tq[row * KC + lane] = cq;
    }
}

// A thread owns four columns and walks a range of rows: sum_i -2 Y_ij c + q g w / alpha_j^2.  Batches of RB rows,
// the next batch's loads in flight and its tables parked in registers, as in skim_scale_grad_kernel.
template <int RB>
struct GradRowsLf {
    uint2 wv[RB];
    float4 gv[RB], yv[RB];
    uint32_t lv[RB];
};

template <int RB>
__device__ __forceinline__ void grad_load_lf(const ScaleLfArgs &b, int64_t rb, int64_t r1, int j0, bool in, GradRowsLf<RB> &r)
{
    const ScaleArgs &a = b.s;
#pragma unroll
    for (int q = 0; q < RB; ++q) {
        const int64_t row = rb + q;
        r.wv[q] = make_uint2(0u, 0u); r.gv[q] = make_float4(0.f, 0.f, 0.f, 0.f); r.yv[q] = r.gv[q]; r.lv[q] = 0u;
        if (row < r1 && in) {
            r.wv[q] = __ldcs(reinterpret_cast<const uint2 *>(a.W + row * a.ld + j0));
            r.gv[q] = __ldcs(reinterpret_cast<const float4 *>(a.G + row * a.ld + j0));
            r.yv[q] = __ldcs(reinterpret_cast<const float4 *>(b.Y + row * (int64_t)a.cols + j0));
            r.lv[q] = __ldcs(reinterpret_cast<const uint32_t *>(a.labels + row * (int64_t)a.cols + j0));
        }
    }
}

__global__ void __launch_bounds__(GT, 2) skim_scale_lf_grad_kernel(ScaleLfArgs b)
{
    constexpr int RB = 2;
    __shared__ double2 tq_s[2][RB * KC];
    const ScaleArgs &a = b.s;
    const int j0 = (blockIdx.x * GT + threadIdx.x) * GC;
    const int64_t r0 = (int64_t)blockIdx.y * a.rows_per_range;
    const int64_t r1 = min(a.rows, r0 + a.rows_per_range);
    const double yscale = ldexp(1.0, -b.exp2);
    double rr[GC], acc[GC];
#pragma unroll
    for (int u = 0; u < GC; ++u) {
        const double al = j0 + u < a.cols ? a.alpha[j0 + u] : 1.0;
        const double r = __drcp_rn(al);
        rr[u] = r * r;
        acc[u] = 0.0;
    }
    const bool in = j0 + GC <= a.cols;           // cols is a multiple of 8: a thread's columns are all inside or all outside
    const bool tq_thread = threadIdx.x < RB * KC;
    GradRowsLf<RB> cur, nxt;
    grad_load_lf<RB>(b, r0, r1, j0, in, cur);
    if (tq_thread && r0 + threadIdx.x / KC < r1) tq_s[0][threadIdx.x] = a.tq[r0 * KC + threadIdx.x];
    int buf = 0;
    for (int64_t rb = r0; rb < r1; rb += RB, buf ^= 1) {
        const int64_t rn = rb + RB;
        double2 tnext = make_double2(0.0, 0.0);
        if (rn < r1) {
            grad_load_lf<RB>(b, rn, r1, j0, in, nxt);
            if (tq_thread && rn + threadIdx.x / KC < r1) tnext = a.tq[rn * KC + threadIdx.x];
        }
        __syncthreads();                        // this batch's tables are in place; the other buffer is no longer read
#pragma unroll
        for (int q = 0; q < RB; ++q) {
            if (rb + q >= r1) break;
            const double2 *tq = tq_s[buf] + q * KC;
            const uint32_t ww[2] = {cur.wv[q].x, cur.wv[q].y};
            const float g[GC] = {cur.gv[q].x, cur.gv[q].y, cur.gv[q].z, cur.gv[q].w};
            const float y[GC] = {cur.yv[q].x, cur.yv[q].y, cur.yv[q].z, cur.yv[q].w};
#pragma unroll
            for (int u = 0; u < GC; ++u) {
                const double2 cq = tq[(cur.lv[q] >> (8 * u)) & (KC - 1)];
                const double wd = (double)__half2float(__ushort_as_half((uint16_t)((u & 1) ? (ww[u >> 1] >> 16) : (ww[u >> 1] & 0xffffu))));
                acc[u] += cq.y * (double)g[u] * wd * rr[u] - 2.0 * ((double)y[u] * yscale) * cq.x;
            }
        }
        if (tq_thread) tq_s[buf ^ 1][threadIdx.x] = tnext;
        cur = nxt;
    }
    if (in) {
#pragma unroll
        for (int u = 0; u < GC; ++u) a.grad_part[(int64_t)blockIdx.y * a.cols + j0 + u] = acc[u];
    }
}

}  // namespace

size_t skim_scale_lfull_scratch_bytes(int64_t rows, int64_t cols)
{
    return skim_align256((size_t)rows * cols * 2) + skim_align256((size_t)rows * cols * 4) + skim_lfull_scratch_bytes(rows, cols);
}

int skim_launch_scale_update_lfull(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                                   int64_t ld, const uint8_t *labels, const uint16_t *H, int64_t ldh, float *alpha,
                                   int steps, float lr0, float decay, int decay_every, int exp2, void *scratch,
                                   double *loss_trace)
{
    SkimWorkspace ws = skim_carve(ctx->ws, rows, cols);
    const unsigned cb = (unsigned)((cols + 255) / 256), ab = (unsigned)((cols + 31) / 32);   // Adam: 32 columns a block
    skim_scale_init_kernel<<<cb, 256, 0, ctx->stream>>>(alpha, (int)cols, ws.alpha64, ws.alpha_il, ws.adam_m, ws.adam_v, ws.status);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    ScaleLfArgs b;
    ScaleArgs &a = b.s;
    a.W = W;
    a.G = importance;
    a.labels = labels;
    a.alpha = ws.alpha64;
    a.alpha_il = ws.alpha_il;
    a.rows = rows;
    a.ld = ld;
    a.cols = (int)cols;
    a.vec = 1;
    a.tconst = reinterpret_cast<double2 *>(ws.scale_const);
    a.tq = reinterpret_cast<double2 *>(ws.scale_cq);
    a.loss_row = ws.loss_part;
    a.grad_part = ws.grad_part;
    unsigned char *sp = (unsigned char *)scratch;
    b.D = (uint16_t *)sp;
    sp += skim_align256((size_t)rows * cols * 2);
    float *Y = (float *)sp;
    sp += skim_align256((size_t)rows * cols * 4);
    void *gemm_scratch = sp;
    b.Y = Y;
    b.exp2 = exp2;
    const int tiles = (int)((cols + GT * GC - 1) / (GT * GC));
    int ranges = (4 * ctx->sm_count + tiles - 1) / tiles;
    if (ranges > SKIM_SCALE_MAX_CTAS) ranges = SKIM_SCALE_MAX_CTAS;
    if (ranges > rows) ranges = (int)rows;
    a.rows_per_range = (int)((rows + ranges - 1) / ranges);
    ranges = (int)((rows + a.rows_per_range - 1) / a.rows_per_range);
    const size_t smem_init = (size_t)SW * NSUM * KC * 32 * sizeof(double);
    const size_t smem_res = (size_t)SW * KC * 32 * sizeof(double) + (size_t)SW * KC * sizeof(double);
    const size_t smem_r = (size_t)SW * KC * 32 * sizeof(double);
    const unsigned sum_blocks = (unsigned)((rows + SW - 1) / SW);
    SKIM_CUDA_OK(cudaFuncSetAttribute(skim_scale_sums_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_init));
    skim_scale_sums_kernel<true, true><<<sum_blocks, SW * 32, smem_init, ctx->stream>>>(a);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    const double beta1 = 0.9, beta2 = 0.999, eps = 1e-8;
    double p1 = 1.0, p2 = 1.0, lr = (double)lr0;
    for (int t = 0; t < steps; ++t) {
        if (t > 0 && t % decay_every == 0) lr *= (double)decay;
        p1 *= beta1;
        p2 *= beta2;
        skim_scale_lf_residual_kernel<<<sum_blocks, SW * 32, smem_res, ctx->stream>>>(b);
        SKIM_CUDA_OK(cudaGetLastError());
        ctx->launches += 1;
        const int rc = skim_launch_err_lfull(ctx, b.D, rows, cols, cols, H, ldh, exp2, gemm_scratch, nullptr, 1, Y, cols, ws.loss_part);
        if (rc) return rc;
        skim_scale_lf_r_kernel<<<sum_blocks, SW * 32, smem_r, ctx->stream>>>(b);
        SKIM_CUDA_OK(cudaGetLastError());
        skim_scale_lf_grad_kernel<<<dim3((unsigned)tiles, (unsigned)ranges), GT, 0, ctx->stream>>>(b);
        SKIM_CUDA_OK(cudaGetLastError());
        skim_scale_adam_kernel<<<ab + 1, 256, 0, ctx->stream>>>(ws.grad_part, ws.loss_part, ranges, rows, (int)cols,
                                                                ws.alpha64, ws.alpha_il, ws.adam_m, ws.adam_v, lr, beta1,
                                                                beta2,
                                                                1.0 - p1, 1.0 - p2, eps,
                                                                loss_trace ? loss_trace + t : nullptr);
        SKIM_CUDA_OK(cudaGetLastError());
        ctx->launches += 3;
    }
    skim_scale_finish_kernel<<<cb, 256, 0, ctx->stream>>>(ws.alpha64, (int)cols, alpha);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}

int skim_launch_scale_update(skim_ctx *ctx, const uint16_t *W, const float *importance, int64_t rows, int64_t cols,
                             int64_t ld, const uint8_t *labels, float *alpha, int steps, float lr0, float decay,
                             int decay_every, double *loss_trace)
{
    SkimWorkspace ws = skim_carve(ctx->ws, rows, cols);
    const unsigned cb = (unsigned)((cols + 255) / 256), ab = (unsigned)((cols + 31) / 32);   // Adam: 32 columns a block
    skim_scale_init_kernel<<<cb, 256, 0, ctx->stream>>>(alpha, (int)cols, ws.alpha64, ws.alpha_il, ws.adam_m, ws.adam_v, ws.status);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    ScaleArgs a;
    a.W = W;
    a.G = importance;
    a.labels = labels;
    a.alpha = ws.alpha64;
    a.alpha_il = ws.alpha_il;
    a.rows = rows;
    a.ld = ld;
    a.cols = (int)cols;
    a.vec = ((reinterpret_cast<uintptr_t>(W) & 15u) == 0 && (reinterpret_cast<uintptr_t>(importance) & 15u) == 0 &&
             (reinterpret_cast<uintptr_t>(labels) & 7u) == 0 && ld % 8 == 0 && cols % 8 == 0) ? 1 : 0;
    a.tconst = reinterpret_cast<double2 *>(ws.scale_const);
    a.tq = reinterpret_cast<double2 *>(ws.scale_cq);
    a.loss_row = ws.loss_part;
    a.grad_part = ws.grad_part;
    // gradient kernel: column tiles x row ranges, about four blocks per SM in all
    const int tiles = (int)((cols + GT * GC - 1) / (GT * GC));
    int ranges = (4 * ctx->sm_count + tiles - 1) / tiles;
    if (ranges > SKIM_SCALE_MAX_CTAS) ranges = SKIM_SCALE_MAX_CTAS;
    if (ranges > rows) ranges = (int)rows;
    a.rows_per_range = (int)((rows + ranges - 1) / ranges);
    ranges = (int)((rows + a.rows_per_range - 1) / a.rows_per_range);
    const size_t smem = (size_t)SW * NSUM * KC * 32 * sizeof(double);
    const unsigned sum_blocks = (unsigned)((rows + SW - 1) / SW);
    auto sums_init = a.vec ? skim_scale_sums_kernel<true, true> : skim_scale_sums_kernel<true, false>;
    auto sums_step = a.vec ? skim_scale_sums_kernel<false, true> : skim_scale_sums_kernel<false, false>;
    auto grad = a.vec ? skim_scale_grad_kernel<true> : skim_scale_grad_kernel<false>;
    SKIM_CUDA_OK(cudaFuncSetAttribute(sums_init, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    SKIM_CUDA_OK(cudaFuncSetAttribute(sums_step, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    sums_init<<<sum_blocks, SW * 32, smem, ctx->stream>>>(a);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    const double beta1 = 0.9, beta2 = 0.999, eps = 1e-8;
    double p1 = 1.0, p2 = 1.0, lr = (double)lr0;
    for (int t = 0; t < steps; ++t) {
        if (t > 0 && t % decay_every == 0) lr *= (double)decay;
        p1 *= beta1;
        p2 *= beta2;
        sums_step<<<sum_blocks, SW * 32, smem, ctx->stream>>>(a);
        SKIM_CUDA_OK(cudaGetLastError());
        grad<<<dim3((unsigned)tiles, (unsigned)ranges), GT, 0, ctx->stream>>>(a);
        SKIM_CUDA_OK(cudaGetLastError());
        skim_scale_adam_kernel<<<ab + 1, 256, 0, ctx->stream>>>(ws.grad_part, ws.loss_part, ranges, rows, (int)cols,
                                                                ws.alpha64, ws.alpha_il, ws.adam_m, ws.adam_v, lr, beta1,
                                                                beta2,
                                                                1.0 - p1, 1.0 - p2, eps,
                                                                loss_trace ? loss_trace + t : nullptr);
        SKIM_CUDA_OK(cudaGetLastError());
        ctx->launches += 3;
    }
    skim_scale_finish_kernel<<<cb, 256, 0, ctx->stream>>>(ws.alpha64, (int)cols, alpha);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
