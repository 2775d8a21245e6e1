// Exact 1-D weighted K-means of every row: the optimum of the clustering objective of SKIM Section 3.2
// (diagonal form), sum_j g_j (x_j - c_{l_j})^2, which the Lloyd iterations of Algorithm 3 only approach.
// In one dimension the optimal clusters are intervals of the sorted row, so the optimum is a dynamic programme
// over split points,
//     F_1(i) = cost(0, i),    F_j(i) = min_{j-1 <= t < i} F_{j-1}(t) + cost(t, i),
//     cost(t, i) = S2 - S1^2 / S0 over the sorted elements t .. i-1 (0 for an interval without weight),
// and the minimising t never decreases with i, which turns the quadratic search of a layer into m log m
// evaluations.  One block owns a row and reads the row record the sort kernels leave (sorted values and
// importances by groups of 8 with their binary64 prefix sums).
//
//   prefix   the record's two-level prefix sums become one flat array Q[t] = (P0, P1, P2, F_{j-1})(t): a cost
//            evaluation is one 32-byte load.
//   layer    positions are visited like the in-order nodes of a perfect binary tree, level by level: a node's
//            search range is bounded by the minimisers of its two nearest finished neighbours.  The first
//            levels have few nodes with long ranges (a group of threads shares a node and reduces), the last
//            ones many nodes with short ranges (one thread per node).
//   result   for every width the split points are walked back from the row's end; centroid = weighted mean of
//            its interval (an interval without weight: mean of its first and last value), error = F_k(m).
// All widths share the layers: F_2, F_4, F_8, F_16 are read off on the way.
#include "skim_cluster_phases.cuh"

namespace {

using namespace skimk;

constexpr int XT = 256;                       // threads per block
constexpr int X_MAX_K = 1 << SKIM_MAX_BIT;    // 16 layers at most

struct ExactSlot {
    size_t q, fc, t, total;                   // byte offsets inside a block's scratch slot
};

__host__ __device__ inline ExactSlot exact_slot(int m)
{
    ExactSlot S;
    const size_t mpad = ((size_t)m + 7) & ~(size_t)7;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += (b + 255) & ~(size_t)255; return o; };
    S.q = take((mpad + 8) * 32);                                  // double4 per position 0 .. mpad
    S.fc = take(((size_t)m + 1) * 8);                             // the layer being filled
    S.t = take((size_t)(X_MAX_K + 1) * ((size_t)m + 1) * 2);      // minimisers of every layer, 16-bit
    S.total = off;
    return S;
}

__device__ __forceinline__ double4 ld_q(const double4 *p)
{
    double4 v;
    asm volatile("ld.global.v4.f64 {%0, %1, %2, %3}, [%4];" : "=d"(v.x), "=d"(v.y), "=d"(v.z), "=d"(v.w) : "l"(p));
    return v;
}

// cost of the interval [t, i) given Q[t] and Q[i]
__device__ __forceinline__ double interval_cost(const double4 &qt, const double4 &qi)
{
    const double s0 = qi.x - qt.x, s1 = qi.y - qt.y, s2 = qi.z - qt.z;
    return s0 > 0.0 ? s2 - s1 * s1 / s0 : 0.0;
}

__global__ void __launch_bounds__(XT) skim_exact_kernel(ClusterArgs a, int rows_in_chunk, unsigned char *scratch, size_t slot_bytes)
{
    extern __shared__ __align__(16) unsigned char xsmem[];
    __shared__ double sval[XT];
    __shared__ int sarg[XT];
    __shared__ float s_dvals[16];
    const int tid = threadIdx.x;
    const int m = a.m;
    const RowRecord R = row_record(m);
    const ExactSlot S = exact_slot(m);
    unsigned char *slot = scratch + (size_t)blockIdx.x * slot_bytes;
    double4 *Q = reinterpret_cast<double4 *>(slot + S.q);
    double *Fc = reinterpret_cast<double *>(slot + S.fc);
    uint16_t *T = reinterpret_cast<uint16_t *>(slot + S.t);
    uint16_t *optarr = reinterpret_cast<uint16_t *>(xsmem);           // minimisers of the current layer by node position
    const int kmax = 1 << (a.bmin + a.nb - 1);

    for (int local = blockIdx.x; local < rows_in_chunk; local += gridDim.x) {
        const int64_t row = a.row0 + local;
        const unsigned char *rec = a.scratch + (size_t)local * (size_t)a.rec_stride;
        const int nd_rec = *reinterpret_cast<const int *>(rec);
        if (nd_rec < 0) continue;                                   // the sort kernel gave the row up
        const int nd = max(nd_rec, 1);
        if (tid < 16) s_dvals[tid] = reinterpret_cast<const float *>(rec + 64)[tid];
        const unsigned char *groups = rec + R.groups;
        const double4 *seg = reinterpret_cast<const double4 *>(rec + R.seg);

        // ------------------------------------------------------------ flat prefix sums
        for (int q = tid; q < R.ngrp; q += XT) {
            const unsigned char *gr = groups + (size_t)q * SKIM_GROUP_BYTES;
            const float4 xa = *reinterpret_cast<const float4 *>(gr), xb = *reinterpret_cast<const float4 *>(gr + 16);
            const float4 ga = *reinterpret_cast<const float4 *>(gr + 32), gb = *reinterpret_cast<const float4 *>(gr + 48);
            const double4 gp = *reinterpret_cast<const double4 *>(gr + 64);
            const double4 sb = seg[q >> SKIM_SEG_SHIFT];
            double p0 = sb.x + gp.x, p1 = sb.y + gp.y, p2 = sb.z + gp.z;
            const float xs[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
            const float gs[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                Q[q * 8 + u] = make_double4(p0, p1, p2, 0.0);
                const double g = (double)gs[u], x = (double)xs[u];      // padding: g = 0
                p0 += g;
                p1 += g * x;
                p2 += g * x * x;
            }
            if (q == R.ngrp - 1) Q[q * 8 + 8] = make_double4(p0, p1, p2, 0.0);
        }
        __syncthreads();

        // ------------------------------------------------------------ layer 1
        const double4 q0 = ld_q(Q);
        for (int i = 1 + tid; i <= m; i += XT) {
            double4 qi = ld_q(Q + i);
            qi.w = interval_cost(q0, qi);
            Q[i] = qi;
        }
        __syncthreads();

        // ------------------------------------------------------------ layers 2 .. kmax
        const int layers = min(min(kmax, nd - 1), m);         // widths with k >= nd take the distinct values instead
        for (int j = 2; j <= layers; ++j) {
            const int n = m - j + 1;                           // positions p = 1 .. n  <->  i = j + p - 1
            int L = 1;
            while ((1 << L) - 1 < n) ++L;
            if (tid == 0) optarr[0] = (uint16_t)(j - 1);
            __syncthreads();
            for (int lev = 0; lev < L; ++lev) {
                const int h = 1 << (L - 1 - lev);
                const int nodes = 1 << lev;
                if (nodes <= XT) {
                    // a group of G threads per node
                    const int G = XT >> lev;
                    const int qn = tid / G, r = tid - qn * G;
                    const int p = (2 * qn + 1) * h;
                    double best = __longlong_as_double(0x7ff0000000000000ll);     // +inf
                    int bt = 0x7fffffff;
                    int i = 0;
                    if (p <= n) {
                        i = j + p - 1;
                        const int tlo = optarr[p - h];
                        int thi = i - 1;
                        if (p + h <= n) thi = min(thi, (int)optarr[p + h]);
                        thi = max(thi, tlo);                   // rounding may break the ordering of two near-tied minimisers
                        const double4 qi = ld_q(Q + i);
                        for (int t = tlo + r; t <= thi; t += G) {
                            const double4 qt = ld_q(Q + t);
                            const double v = qt.w + interval_cost(qt, qi);
                            if (v < best) { best = v; bt = t; }
                        }
                    }
                    if (G > 1) {
                        sval[tid] = best;
                        sarg[tid] = bt;
                        __syncthreads();
                        for (int s = G >> 1; s >= 1; s >>= 1) {
                            if (r < s) {
                                const double ov = sval[tid + s];
                                const int ot = sarg[tid + s];
                                if (ov < best || (ov == best && ot < bt)) { best = ov; bt = ot; }
                                sval[tid] = best;
                                sarg[tid] = bt;
                            }
                            __syncthreads();
                        }
                    }
                    if (r == 0 && p <= n) {
                        optarr[p] = (uint16_t)bt;
                        Fc[i] = best;
                        T[(size_t)j * (m + 1) + i] = (uint16_t)bt;
                    }
                } else {
                    for (int qn = tid; qn < nodes; qn += XT) {
                        const int p = (2 * qn + 1) * h;
                        if (p > n) break;
                        const int i = j + p - 1;
                        const int tlo = optarr[p - h];
                        int thi = i - 1;
                        if (p + h <= n) thi = min(thi, (int)optarr[p + h]);
                        thi = max(thi, tlo);
                        const double4 qi = ld_q(Q + i);
                        double best = __longlong_as_double(0x7ff0000000000000ll);
                        int bt = tlo;
                        for (int t = tlo; t <= thi; ++t) {
                            const double4 qt = ld_q(Q + t);
                            const double v = qt.w + interval_cost(qt, qi);
                            if (v < best) { best = v; bt = t; }
                        }
                        optarr[p] = (uint16_t)bt;
                        Fc[i] = best;
                        T[(size_t)j * (m + 1) + i] = (uint16_t)bt;
                    }
                }
                __syncthreads();
            }
            // F_j becomes the previous layer
            for (int i = j + tid; i <= m; i += XT) {
                const double f = Fc[i];
                reinterpret_cast<double *>(Q + i)[3] = f;
            }
            __syncthreads();
        }

        // ------------------------------------------------------------ results, one thread per width
        if (tid < a.nb) {
            const int width = a.bmin + tid;
            const int k = 1 << width;
            int off = 0;
            for (int u = 0; u < tid; ++u) off += 1 << (a.bmin + u);
            float *cout = a.centroids + row * a.sumk + off;
            if (nd <= k) {
                for (int u = 0; u < k; ++u) cout[u] = s_dvals[min(u, nd - 1)];
                a.err[row * a.nb + tid] = 0.0f;
            } else {
                // F_k(m) was overwritten by later layers in Q; walk the minimisers back and add the interval costs up
                int i = m;
                double total = 0.0;
                for (int jj = k; jj >= 1; --jj) {
                    const int t = (jj == 1) ? 0 : (int)T[(size_t)jj * (m + 1) + i];
                    const double4 qi = ld_q(Q + i), qt = ld_q(Q + t);
                    const double s0 = qi.x - qt.x;
                    float c;
                    if (s0 > 0.0) {
                        c = (float)((qi.y - qt.y) / s0);
                    } else {
                        const float xf = *(reinterpret_cast<const float *>(groups + (size_t)(t >> 3) * SKIM_GROUP_BYTES) + (t & 7));
                        const float xl = *(reinterpret_cast<const float *>(groups + (size_t)((i - 1) >> 3) * SKIM_GROUP_BYTES) + ((i - 1) & 7));
                        c = (float)(0.5 * ((double)xf + (double)xl));
                    }
                    cout[jj - 1] = c;
                    total += interval_cost(qt, qi);
                    i = t;
                }
                a.err[row * a.nb + tid] = (float)fmax(total, 0.0);
            }
        }
        __syncthreads();
    }
}

}  // namespace

size_t skim_exact_slot_bytes(int64_t cols) { return exact_slot((int)cols).total; }

int skim_exact_slots(const skim_ctx *ctx, int64_t rows)
{
    const int64_t want = (int64_t)ctx->sm_count * 3;
    return (int)(rows < want ? rows : want);
}

int skim_launch_exact(skim_ctx *ctx, const ClusterArgs &args, int64_t rows, void *scratch, int slots)
{
    int L = 1;
    while ((1 << L) - 1 < args.m) ++L;
    const size_t smem = ((size_t)(1 << L) + 8) * sizeof(uint16_t);
    if (smem > (size_t)ctx->max_smem_optin) return SKIM_ERR_SHAPE;
    SKIM_CUDA_OK(cudaFuncSetAttribute(skim_exact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const unsigned blocks = (unsigned)(rows < slots ? rows : slots);
    skim_exact_kernel<<<blocks, XT, smem, ctx->stream>>>(args, (int)rows, (unsigned char *)scratch, exact_slot(args.m).total);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
