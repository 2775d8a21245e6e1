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
//            search range is bounded by the minimisers of its two nearest finished neighbours.  The ranges of
//            a level tile the span of split points; the span is dealt to the threads in equal stretches and
//            the candidates of a node meet in one atomic minimum, because the ranges themselves are very
//            unequal (the minimiser jumps where an outlier enters the prefix).
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

// shared memory: the minimisers by tree position (2^L + 8 entries, 2^L - 1 >= m), then one key per node of a level
__host__ __device__ inline size_t exact_optarr_bytes(int m)
{
    int L = 1;
    while ((1 << L) - 1 < m) ++L;
    return ((((size_t)1 << L) + 8) * sizeof(uint16_t) + 15) & ~(size_t)15;
}
__host__ __device__ inline size_t exact_smem_bytes(int m) { return exact_optarr_bytes(m) + ((size_t)m / 2 + 8) * sizeof(unsigned long long); }

__device__ __forceinline__ double4 ld_q(const double4 *p)
{
    double4 v;
    asm volatile("ld.global.v4.f64 {%0, %1, %2, %3}, [%4];" : "=d"(v.x), "=d"(v.y), "=d"(v.z), "=d"(v.w) : "l"(p));
    return v;
}

// Candidates of one node compete through a 64-bit atomic minimum: the order-preserving image of the cost with
// its 16 lowest mantissa bits replaced by the split point, so that costs equal to 2^-36 relative go to the
// smaller split point.
__device__ __forceinline__ unsigned long long candidate_key(double v, int t)
{
    if (v == 0.0) v = 0.0;
    const unsigned long long u = (unsigned long long)__double_as_longlong(v);
    const unsigned long long ob = (u >> 63) ? ~u : (u | 0x8000000000000000ull);
    return (ob & ~0xffffull) | (unsigned long long)(unsigned)t;
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
    unsigned long long *keys = reinterpret_cast<unsigned long long *>(xsmem + exact_optarr_bytes(m));   // per node of a level
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
                const int nvalid = (n / h + 1) >> 1;                 // nodes (2q + 1) h <= n of this level
                // a node's position, and the range of split points its two finished neighbours leave it
                auto node_i = [&](int q) { return j + (2 * q + 1) * h - 1; };
                auto node_tlo = [&](int q) { return (int)optarr[2 * q * h]; };
                auto node_thi = [&](int q) {
                    const int i = node_i(q);
                    int thi = i - 1;
                    if ((2 * q + 2) * h <= n) thi = min(thi, (int)optarr[(2 * q + 2) * h]);
                    return max(thi, node_tlo(q));                   // rounding may break the order of two near-tied minimisers
                };
                for (int q = tid; q < nvalid; q += XT) keys[q] = ~0ull;
                __syncthreads();
                // The ranges of a level's nodes tile the span of split points, sharing their end points.  The
                // span, not the nodes, is dealt to the threads in equal stretches (a node's range can be a
                // thousand times another's); a thread walks its stretch node by node and commits each node's
                // best candidate with one atomic minimum on (cost rounded to 2^-36 relative, split point).
                const int tmin = (int)optarr[0], tmax = node_thi(nvalid - 1);
                const int chunk = (tmax - tmin + XT) / XT;
                const int ta = tmin + tid * chunk, tb = min(ta + chunk, tmax + 1);
                if (ta < tb) {
                    int lo = 0, hi = nvalid - 1;
                    while (lo < hi) {
                        const int mid = (lo + hi) >> 1;
                        if (node_thi(mid) < ta) lo = mid + 1; else hi = mid;
                    }
                    for (int q = lo; q < nvalid; ++q) {
                        const int tlo = node_tlo(q), thi = node_thi(q);
                        if (tlo >= tb) break;
                        const int t0 = max(ta, tlo), t1 = min(tb - 1, thi);
                        if (t0 <= t1) {
                            const double4 qi = ld_q(Q + node_i(q));
                            double best = __longlong_as_double(0x7ff0000000000000ll);     // +inf
                            int bt = t0;
                            int t = t0;
                            for (; t + 3 <= t1; t += 4) {            // four loads in flight
                                const double4 qa = ld_q(Q + t), qb = ld_q(Q + t + 1), qc = ld_q(Q + t + 2), qd = ld_q(Q + t + 3);
                                const double va = qa.w + interval_cost(qa, qi), vb = qb.w + interval_cost(qb, qi);
                                const double vc = qc.w + interval_cost(qc, qi), vd = qd.w + interval_cost(qd, qi);
                                if (va < best) { best = va; bt = t; }
                                if (vb < best) { best = vb; bt = t + 1; }
                                if (vc < best) { best = vc; bt = t + 2; }
                                if (vd < best) { best = vd; bt = t + 3; }
                            }
                            for (; t <= t1; ++t) {
                                const double4 qt = ld_q(Q + t);
                                const double v = qt.w + interval_cost(qt, qi);
                                if (v < best) { best = v; bt = t; }
                            }
                            atomicMin(&keys[q], candidate_key(best, bt));
                        }
                        if (thi >= tb) break;                        // the rest of this node, and all later ones, are other threads'
                    }
                }
                __syncthreads();
                for (int q = tid; q < nvalid; q += XT) {
                    const int i = node_i(q);
                    const double4 qi = ld_q(Q + i);
                    const unsigned long long key = keys[q];
                    int bt = (int)(key & 0xffffull);
                    double best;
                    if (key != ~0ull) {
                        const double4 qt = ld_q(Q + bt);
                        best = qt.w + interval_cost(qt, qi);
                    } else {
                        // no stretch met the node (possible only where rounding broke the order of the ranges)
                        best = __longlong_as_double(0x7ff0000000000000ll);
                        bt = node_tlo(q);
                        for (int t = node_tlo(q); t <= node_thi(q); ++t) {
                            const double4 qt = ld_q(Q + t);
                            const double v = qt.w + interval_cost(qt, qi);
                            if (v < best) { best = v; bt = t; }
                        }
                    }
                    Fc[i] = best;
                    T[(size_t)j * (m + 1) + i] = (uint16_t)bt;
                }
                __syncthreads();
                for (int q = tid; q < nvalid; q += XT) optarr[(2 * q + 1) * h] = T[(size_t)j * (m + 1) + node_i(q)];
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
    const size_t smem = exact_smem_bytes(args.m);
    if (smem > (size_t)ctx->max_smem_optin) return SKIM_ERR_SHAPE;
    SKIM_CUDA_OK(cudaFuncSetAttribute(skim_exact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // as many blocks as are resident at once (each owns a scratch slot), at most `slots`
    int per_sm = 1;
    SKIM_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, skim_exact_kernel, XT, smem));
    int64_t resident = (int64_t)(per_sm > 0 ? per_sm : 1) * ctx->sm_count;
    if (resident > slots) resident = slots;
    const unsigned blocks = (unsigned)(rows < resident ? rows : resident);
    skim_exact_kernel<<<blocks, XT, smem, ctx->stream>>>(args, (int)rows, (unsigned char *)scratch, exact_slot(args.m).total);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
